"""Seeded synthetic inputs (host side, numpy only).

This module serves both the CUDA path and the CPU oracle.  It holds no
arithmetic of the method itself (no packing, no products): only a counter-based
random number generator and the recipes that turn it into coordinate lists and
dense operands shaped like the paper's workloads (Section 6: uniform random
matrices of density 0.01, row-band matrices whose first 1000 rows are dense,
and skewed 3-way tensors standing in for the FROSTT files of Tables 1 and 4).

Generator: splitmix64 evaluated at a counter.  Draw ``k`` of stream ``s`` under
seed ``g`` is ``mix(base(g, s) + (k + 1) * GOLDEN)`` with the published
splitmix64 finaliser ``mix``; every array below is a pure function of
(seed, stream id, index), so any slice can be regenerated anywhere.

All coordinate lists are duplicate free and are returned in a scrambled order
(an affine index permutation), so a packer never sees sorted input.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=_U64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        return z ^ (z >> _U64(31))


def _base(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        a = _mix(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=_U64))
        b = _mix(a + _U64(stream & 0xFFFFFFFFFFFFFFFF) * _GOLDEN + _U64(1))
    return b[0]


def raw_u64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n raw 64-bit draws of (seed, stream), starting at counter ``offset``."""
    idx = np.arange(offset, offset + n, dtype=_U64)
    with np.errstate(over="ignore"):
        return _mix(_base(seed, stream) + (idx + _U64(1)) * _GOLDEN)


def uniform01(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """Uniform doubles in [0, 1) from the top 53 bits."""
    return (raw_u64(seed, stream, n, offset) >> _U64(11)).astype(np.float64) * (1.0 / (1 << 53))


def uniform_pm1(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """Uniform doubles in [-1, 1)."""
    return uniform01(seed, stream, n, offset) * 2.0 - 1.0


def small_ints(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """Non-zero integers in {-4..-1, 1..4} as doubles (exact-arithmetic tests)."""
    r = (raw_u64(seed, stream, n, offset) >> _U64(33)) % _U64(8)
    v = r.astype(np.int64) - 4
    v[v >= 0] += 1
    return v.astype(np.float64)


def randint(seed: int, stream: int, n: int, hi: int, offset: int = 0) -> np.ndarray:
    """Integers in [0, hi) (plain modulo of a 64-bit draw; bias < 2^-40 here)."""
    return (raw_u64(seed, stream, n, offset) % _U64(hi)).astype(np.int64)


def affine_scramble(n: int, seed: int) -> np.ndarray:
    """A fixed permutation e -> (a*e + b) mod n with gcd(a, n) = 1."""
    if n <= 1:
        return np.zeros(n, dtype=np.int64)
    a = (0x9E3779B1 + 2 * (seed % 1000)) % n
    if a < 2:
        a = 1
    while math.gcd(a, n) != 1:
        a += 1
    b = (0x7F4A7C15 + seed) % n
    e = np.arange(n, dtype=np.uint64)
    return ((e * np.uint64(a) + np.uint64(b)) % np.uint64(n)).astype(np.int64)


def _first_distinct(draw, count: int, batch: int) -> np.ndarray:
    """First ``count`` distinct keys, in draw order, of the stream ``draw(offset, n)``."""
    kept = np.empty(0, dtype=np.uint64)
    offset = 0
    while True:
        fresh = draw(offset, batch)
        offset += batch
        allk = np.concatenate([kept, fresh])
        _, first = np.unique(allk, return_index=True)
        first.sort()
        kept = allk[first]
        if kept.size >= count:
            return kept[:count]


def zipf_cdf(n: int, s: float) -> np.ndarray:
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def zipf_ranks(cdf: np.ndarray, u: np.ndarray) -> np.ndarray:
    """Inverse-CDF sample: rank in [0, n) for uniforms u in [0, 1)."""
    return np.minimum(np.searchsorted(cdf, u, side="right"), cdf.size - 1).astype(np.int64)


@dataclass
class Coo:
    """A duplicate-free coordinate list with logical dims (one array per dim)."""

    dims: tuple
    coords: list
    vals: np.ndarray
    meta: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.vals.size)

    @property
    def rank(self) -> int:
        return len(self.dims)


def _finish(dims, cols, seed, integer_values, meta=None) -> Coo:
    n = cols[0].size
    perm = affine_scramble(n, seed)
    coords = [np.ascontiguousarray(c[perm]) for c in cols]
    vals = small_ints(seed, 900, n) if integer_values else uniform_pm1(seed, 900, n)
    return Coo(tuple(int(d) for d in dims), coords, vals, meta or {})


def dense_operand(seed: int, stream: int, rows: int, cols: int, integer_values: bool = False) -> np.ndarray:
    """Row-major dense matrix, uniform in [-1, 1) (or small integers)."""
    f = small_ints if integer_values else uniform_pm1
    return f(seed, stream, rows * cols).reshape(rows, cols)


# --------------------------------------------------------------------------
# Recipes
# --------------------------------------------------------------------------

def uniform_matrix(m: int, n: int, nnz: int, seed: int = 0, integer_values: bool = False) -> Coo:
    """nnz distinct cells of an m x n matrix, uniform (Section 6.2's uniform
    random shape; density 0.01 at 1024^2 gives about 10,486 entries)."""
    nnz = min(nnz, m * n)
    tot = m * n

    def draw(off, cnt):
        return raw_u64(seed, 1, cnt, off) % _U64(tot)

    keys = _first_distinct(draw, nnz, max(1024, int(nnz * 1.1) + 16)) if nnz else np.empty(0, np.uint64)
    r = (keys // _U64(n)).astype(np.int64)
    c = (keys % _U64(n)).astype(np.int64)
    return _finish((m, n), [r, c], seed, integer_values)


def zipf_row_lengths(m: int, s: float, mean: float, seed: int) -> np.ndarray:
    """Row lengths i.i.d. P(len = k) ~ k^-s on 1..kmax, kmax the smallest cut
    whose mean reaches ``mean``."""
    kmax = 1
    while True:
        k = np.arange(1, kmax + 1, dtype=np.float64)
        w = k ** (-s)
        if (k * w).sum() / w.sum() >= mean or kmax > 1 << 20:
            break
        kmax += 1
    cdf = np.cumsum(w) / w.sum()
    return zipf_ranks(cdf, uniform01(seed, 2, m)) + 1


def powerlaw_rows_matrix(m: int, n: int, s: float = 1.5, mean: float = 16.0, seed: int = 0,
                         integer_values: bool = False) -> Coo:
    """Row lengths truncated Zipf(s) with the given mean, columns uniform and
    distinct within a row."""
    lens = np.minimum(zipf_row_lengths(m, s, mean, seed), n)
    rows = np.repeat(np.arange(m, dtype=np.int64), lens)
    cols = randint(seed, 3, rows.size, n)
    rnd = 0
    while True:
        key = rows.astype(np.uint64) * _U64(n) + cols.astype(np.uint64)
        order = np.argsort(key, kind="stable")
        ks = key[order]
        dup = np.zeros(key.size, dtype=bool)
        dup[order[1:]] = ks[1:] == ks[:-1]
        ndup = int(dup.sum())
        if ndup == 0:
            break
        rnd += 1
        cols[dup] = randint(seed, 100 + rnd, ndup, n)
    return _finish((m, n), [rows, cols], seed, integer_values, {"max_row": int(lens.max())})


def confined_rows_matrix(m: int, n: int, nnz: int, row_fraction: float = 0.1, seed: int = 0,
                         integer_values: bool = False) -> Coo:
    """nnz distinct cells whose rows come from a random subset holding
    ``row_fraction`` of all rows; columns uniform."""
    nrows = max(1, int(math.ceil(m * row_fraction)))
    chosen = _first_distinct(lambda off, cnt: raw_u64(seed, 4, cnt, off) % _U64(m), nrows,
                             max(1024, int(nrows * 1.2))).astype(np.int64)
    nnz = min(nnz, nrows * n)

    def draw(off, cnt):
        a = raw_u64(seed, 5, cnt, off) % _U64(nrows)
        b = raw_u64(seed, 6, cnt, off) % _U64(n)
        return a * _U64(n) + b

    keys = _first_distinct(draw, nnz, max(1024, int(nnz * 1.05) + 16))
    r = chosen[(keys // _U64(n)).astype(np.int64)]
    c = (keys % _U64(n)).astype(np.int64)
    return _finish((m, n), [r, c], seed, integer_values, {"rows_used": nrows})


def row_band_matrix(n: int, dense_rows: int = 1000, seed: int = 0, integer_values: bool = False) -> Coo:
    """n x n matrix whose first ``dense_rows`` rows are full (Section 6.2,
    Table 3's input shape); all other rows are empty."""
    dense_rows = min(dense_rows, n)
    e = np.arange(dense_rows * n, dtype=np.int64)
    return _finish((n, n), [e // n, e % n], seed, integer_values)


def zipf_tensor3(dim: int, nnz: int, s: float = 1.2, seed: int = 0, integer_values: bool = False) -> Coo:
    """dim^3 tensor; each mode's coordinate is Zipf(s) over a random relabelling
    of 0..dim-1; the first nnz distinct triples in draw order are kept."""
    nnz = min(nnz, dim ** 3)
    cdf = zipf_cdf(dim, s)
    relabel = [np.argsort(raw_u64(seed, 10 + d, dim), kind="stable").astype(np.int64) for d in range(3)]
    D = _U64(dim)

    def draw(off, cnt):
        k = np.zeros(cnt, dtype=np.uint64)
        for d in range(3):
            c = relabel[d][zipf_ranks(cdf, uniform01(seed, 20 + d, cnt, off))]
            k = k * D + c.astype(np.uint64)
        return k

    keys = _first_distinct(draw, nnz, max(1024, int(nnz * 0.75) + 16)) if nnz else np.empty(0, np.uint64)
    k = (keys % D).astype(np.int64)
    j = ((keys // D) % D).astype(np.int64)
    i = (keys // (D * D)).astype(np.int64)
    return _finish((dim, dim, dim), [i, j, k], seed, integer_values)


def uniform_tensor(dims, nnz: int, seed: int = 0, integer_values: bool = False) -> Coo:
    """nnz distinct uniform cells of a tensor of any rank (small tests)."""
    tot = 1
    for d in dims:
        tot *= int(d)
    nnz = min(nnz, tot)
    keys = _first_distinct(lambda off, cnt: raw_u64(seed, 7, cnt, off) % _U64(tot), nnz,
                           max(64, 2 * nnz)) if nnz else np.empty(0, np.uint64)
    cols = []
    rem = keys.copy()
    for d in reversed(dims):
        cols.append((rem % _U64(d)).astype(np.int64))
        rem = rem // _U64(d)
    cols.reverse()
    return _finish(tuple(dims), cols, seed, integer_values)


# --------------------------------------------------------------------------
# The five benchmark configurations (and the row band used for SpMV timing).
# ``scale`` < 1 shrinks sizes for tests; 1.0 gives the stated sizes.
# --------------------------------------------------------------------------

def config1(seed: int = 0, n: int = 1024, density: float = 0.01, **kw) -> Coo:
    return uniform_matrix(n, n, int(math.ceil(n * n * density)), seed, **kw)


def config2(seed: int = 0, n: int = 65536, **kw) -> Coo:
    return powerlaw_rows_matrix(n, n, 1.5, 16.0, seed, **kw)


def config3(seed: int = 0, n: int = 1 << 20, nnz: int = 5_000_000, **kw) -> Coo:
    return confined_rows_matrix(n, n, nnz, 0.1, seed, **kw)


def config4(seed: int = 0, n: int = 131072, nnz: int = 2_000_000, **kw) -> Coo:
    return uniform_matrix(n, n, nnz, seed, **kw)


def config5(seed: int = 0, dim: int = 16384, nnz: int = 20_000_000, **kw) -> Coo:
    return zipf_tensor3(dim, nnz, 1.2, seed, **kw)


def config1b(seed: int = 0, n: int = 65536, dense_rows: int = 1000, **kw) -> Coo:
    return row_band_matrix(n, dense_rows, seed, **kw)
