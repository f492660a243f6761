"""Seeded random shapes, patterns, encodings, index widths and operand widths: every call of the
path against the oracle (structure bit for bit, values within 1e-12 * sum|a*b|)."""
import numpy as np
import pytest

from gpu_util import assert_close, assert_storage_equal, dev, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu

WIDTHS = [(32, 32, 32), (64, 64, 64), (32, 64, 32), (0, 0, 64)]      # posBits, crdBits, coordinate bits of the input


def _matrix(rng, seed):
    kind = int(rng.integers(0, 5))
    m, n = int(rng.integers(1, 3000)), int(rng.integers(1, 3000))
    nnz = int(rng.integers(0, min(m * n, 60000) + 1))
    if kind == 0:
        return I.uniform_matrix(m, n, nnz, seed)
    if kind == 1:
        return I.powerlaw_rows_matrix(m, n, 1.5, float(rng.uniform(1, min(n, 30))), seed)
    if kind == 2:
        return I.confined_rows_matrix(m, n, min(nnz, max(1, m // 10) * n), 0.1, seed)
    if kind == 3:                                   # duplicate coordinates
        c = I.uniform_matrix(m, n, nnz, seed)
        if c.nnz > 3:
            k = int(rng.integers(1, c.nnz))
            c = I.Coo(c.dims, [np.concatenate([x, x[:k]]) for x in c.coords], np.concatenate([c.vals, c.vals[:k] * 0.5]))
        return c
    m = int(rng.integers(1, 40))                    # few, long rows
    return I.uniform_matrix(m, n, min(nnz, m * n), seed)


@pytest.mark.parametrize("block", range(4))
def test_random_matrices(oracle, block):
    rng = np.random.default_rng(1000 + block)
    for _ in range(12):
        seed = int(rng.integers(1, 1 << 30))
        c = _matrix(rng, seed)
        m, n = c.dims
        lt = tuple(int(x) for x in rng.integers(0, 2, 2))
        od = (0, 1) if rng.random() < 0.5 else (1, 0)
        if lt[1] == 0:                              # dense inner level: only when the slices fit
            stored = c.dims[od[0]] if lt[0] == 0 else np.unique(c.coords[od[0]]).size
            if stored * c.dims[od[1]] > 1 << 22:
                lt = (lt[0], 1)
        pb, cb, cbits = WIDTHS[int(rng.integers(0, len(WIDTHS)))]
        what = f"{c.dims} nnz={c.nnz} lt={lt} ord={od} widths={pb}/{cb}/{cbits} seed={seed}"
        coords, vals = to_dev(c, cbits)
        A = sp().sp_pack(c.dims, coords, vals, lt, od, pb, cb)
        ref = oracle.pack(c.dims, c.coords, c.vals, lt, od)
        assert_storage_equal(A, ref)
        x = I.uniform_pm1(seed, 2, n)
        yr, yb = oracle.spmv(m, c.coords[0], c.coords[1], c.vals, x)
        assert_close(sp().sp_spmv(A, dev(x)).cpu().numpy(), yr, yb, "spmv " + what)
        N = int(rng.choice([1, 2, 3, 7, 16, 32, 33, 48, 64, 70]))
        B = I.dense_operand(seed, 3, n, N)
        Cr, Cb = oracle.spmm(m, c.coords[0], c.coords[1], c.vals, B)
        assert_close(sp().sp_spmm(A, dev(B)).cpu().numpy(), Cr, Cb, f"spmm N={N} " + what)
        K = int(rng.choice([1, 5, 32, 64, 100, 128]))
        Ad, Bd = I.dense_operand(seed, 8, m, K), I.dense_operand(seed, 9, K, n)
        (si, sj), sv = oracle.unpack(ref)           # stored cells in storage order (explicit zeros included)
        if sv.size:
            xr, xb = oracle.sddmm(si, sj, sv, Ad, Bd)
            assert_close(sp().sp_sddmm(A, dev(Ad), dev(Bd)).cpu().numpy(), xr, xb, f"sddmm K={K} " + what)
        oc, ov = sp().sp_unpack(A)
        assert np.array_equal(oc[0].cpu().numpy(), si) and np.array_equal(oc[1].cpu().numpy(), sj)
        assert np.array_equal(ov.cpu().numpy(), sv)


@pytest.mark.parametrize("block", range(3))
def test_random_tensors(oracle, block):
    rng = np.random.default_rng(2000 + block)
    for _ in range(10):
        seed = int(rng.integers(1, 1 << 30))
        dims = tuple(int(x) for x in rng.integers(1, 400, 3))
        nnz = int(rng.integers(0, min(dims[0] * dims[1] * dims[2], 80000) + 1))
        if rng.random() < 0.5 and min(dims) > 20:
            d = int(min(dims))
            c = I.zipf_tensor3(d, min(nnz, d * d * d // 3), 1.2, seed)
        else:
            c = I.uniform_tensor(dims, nnz, seed)
        dims = c.dims
        mode = int(rng.integers(0, 3))
        others = [d for d in range(3) if d != mode]
        if rng.random() < 0.5:
            others = others[::-1]
        od, lt = (mode, others[0], others[1]), (int(rng.integers(0, 2)), 1, 1)
        pb, cb, cbits = WIDTHS[int(rng.integers(0, len(WIDTHS)))]
        R = int(rng.choice([1, 2, 4, 5, 8, 16, 30, 32, 36, 40, 64]))
        what = f"{dims} nnz={c.nnz} lt={lt} ord={od} R={R} widths={pb}/{cb}/{cbits} seed={seed}"
        coords, vals = to_dev(c, cbits)
        T = sp().sp_pack(dims, coords, vals, lt, od, pb, cb)
        assert_storage_equal(T, oracle.pack(dims, c.coords, c.vals, lt, od))
        F = [I.dense_operand(seed, 20 + d, dims[d], R) for d in range(3)]
        rs = sorted(d for d in range(3) if d != mode)
        Mr, Mb = oracle.mttkrp(dims[mode], c.coords[mode], c.coords[rs[0]], c.coords[rs[1]], c.vals, F[rs[0]], F[rs[1]])
        Mg = sp().sp_mttkrp_mode(T, mode, [dev(f) for f in F]).cpu().numpy()
        assert_close(Mg, Mr, Mb, "mttkrp " + what)


def test_random_dense_inner_products(oracle):
    """Row bands and full matrices stored with a dense inner level, random sizes, widths N, paddings of B
    and starts of B on or off a 16-byte boundary: the copy-engine feed and the register-staged feed of
    sp_spmm, chosen by those alignments, against the oracle; what lies beside B and C stays out of it."""
    import torch
    rng = np.random.default_rng(3000)
    for _ in range(24):
        seed = int(rng.integers(1, 1 << 30))
        m, n = int(rng.integers(1, 1500)), int(rng.integers(1, 1500))
        rows = int(rng.integers(1, min(m, 300) + 1))
        N = int(rng.choice([1, 2, 6, 7, 8, 16, 30, 32, 33, 40, 64, 70]))
        ldb, shift = N + int(rng.integers(0, 4)), int(rng.integers(0, 2))
        cdr = rng.random() < 0.7
        cbits = 32 if rng.random() < 0.7 else 64
        rsel = np.sort(rng.choice(m, rows, replace=False)) if cdr else np.arange(m)
        e = np.arange(rsel.size * n, dtype=np.int64)
        coo = I.Coo((m, n), [rsel[e // n], e % n], I.uniform_pm1(seed, 1, e.size))
        B = I.dense_operand(seed, 3, n, N)
        ref, bd = oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B)
        coords, vals = to_dev(coo, cbits)
        A = sp().sp_pack(coo.dims, coords, vals, (1 if cdr else 0, 0), (0, 1), 32, cbits)
        flat = torch.full((n * ldb + 2,), 1e300, dtype=torch.float64, device="cuda")
        Bdev = flat[shift:shift + n * ldb].view(n, ldb)[:, :N]
        Bdev.copy_(dev(B))
        Cbig = torch.full((m, N + 2), 7.0, dtype=torch.float64, device="cuda")
        sp().sp_spmm(A, Bdev, Cbig[:, :N])
        assert_close(Cbig[:, :N].cpu().numpy(), ref, bd, f"dense inner {(m, n, rows, N, ldb, shift, cdr, cbits)}")
        assert torch.all(Cbig[:, N:] == 7.0)
