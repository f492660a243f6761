"""Allocator failures injected on the host through sp_set_allocator: an allocator that returns NULL on
its k-th call, for every k a call reaches.  Each call must answer SP_ERR_ALLOC, give back everything
it had taken, and leave the library usable.  No GPU fault is involved: the failing call is the hook."""
import ctypes as C

import numpy as np
import pytest
import torch

from gpu_util import assert_close, dev, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu

SP_ERR_ALLOC = 6


class FailingAllocator:
    """Hands out torch caching-allocator memory, returns NULL on call number `fail_at` (1-based), and
    keeps the set of live pointers."""

    def __init__(self):
        b = sp()
        self.b = b
        self.calls = 0
        self.fail_at = 0
        self.live = {}
        self.failed = False

        def alloc(nbytes, stream, ctx):
            self.calls += 1
            if self.calls == self.fail_at:
                self.failed = True
                return None
            p = torch.cuda.caching_allocator_alloc(max(int(nbytes), 1), stream=int(stream or 0))
            self.live[p] = nbytes
            return p

        def free(ptr, stream, ctx):
            if ptr:
                assert ptr in self.live, "the library freed a pointer it was never given (or freed it twice)"
                del self.live[ptr]
                torch.cuda.caching_allocator_delete(ptr)

        self._a, self._f = b._ALLOC_T(alloc), b._FREE_T(free)

    def __enter__(self):
        self.b.use_torch_allocator()        # so that the binding does not install its own hook over this one
        assert self.b._lib.sp_set_allocator(self._a, self._f, None) == 0
        return self

    def __exit__(self, *exc):
        torch.cuda.synchronize()
        self.b._lib.sp_set_allocator(self.b._alloc_cb, self.b._free_cb, None)
        self.b._allocator_set = True

    def arm(self, k):
        self.calls, self.fail_at, self.failed = 0, k, False


def sweep(alloc, call, cleanup=lambda r: r.free() if hasattr(r, "free") else None, limit=200):
    """Fails the k-th allocation of `call` for k = 1, 2, ... until the call gets through; returns the
    number of failure points met."""
    points = 0
    for k in range(1, limit):
        before = dict(alloc.live)
        alloc.arm(k)
        try:
            r = call()
        except alloc.b.SpError as e:
            assert alloc.failed and e.code == SP_ERR_ALLOC, f"k={k}: status {e.code}"
            torch.cuda.synchronize()
            assert alloc.live == before, f"k={k}: {len(alloc.live) - len(before)} allocation(s) not given back"
            points += 1
            continue
        assert not alloc.failed, f"k={k}: an allocation failed and the call still reported success"
        cleanup(r)
        torch.cuda.synchronize()
        assert alloc.live == before
        return points
    raise AssertionError("the call never got through")


@pytest.fixture()
def alloc():
    with FailingAllocator() as a:
        yield a
    assert not a.live, "memory still held after every handle was freed"


@pytest.mark.parametrize("lt,od", [((0, 1), (0, 1)), ((1, 1), (0, 1)), ((0, 1), (1, 0)), ((1, 0), (0, 1)), ((0, 0), (0, 1))])
def test_pack_gives_everything_back(alloc, lt, od):
    coo = I.config3(seed=5, n=1 << 10, nnz=6000)
    coords, vals = to_dev(coo)
    pts = sweep(alloc, lambda: sp().sp_pack(coo.dims, coords, vals, lt, od))
    assert pts >= 2          # the pack's workspace (one block), the handle's arrays (one block), scan scratch ...
    alloc.arm(0)
    sp().sp_pack(coo.dims, coords, vals, lt, od).free()     # and the next call works


def test_pack_rank3_and_convert(alloc):
    t = I.config5(seed=5, dim=64, nnz=5000)
    coords, vals = to_dev(t)
    assert sweep(alloc, lambda: sp().sp_pack(t.dims, coords, vals, (0, 1, 1))) >= 2
    alloc.arm(0)
    T = sp().sp_pack(t.dims, coords, vals, (1, 1, 1))
    assert sweep(alloc, lambda: sp().sp_convert(T, (0, 1, 1), (0, 2, 1))) >= 3
    T.free()


def test_compute_calls_give_everything_back(alloc, oracle):
    coo = I.config3(seed=6, n=1 << 10, nnz=6000)
    coords, vals = to_dev(coo)
    B = I.dense_operand(6, 31, coo.dims[1], 8)
    Bd, xd = dev(B), dev(B[:, 0].copy())
    ref, bd = oracle.spmm(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, B)
    out = torch.empty(coo.dims[0], 8, dtype=torch.float64, device="cuda")
    y = torch.empty(coo.dims[0], dtype=torch.float64, device="cuda")
    for lt, od, pb in [((0, 1), (0, 1), 32), ((1, 1), (0, 1), 32), ((0, 1), (1, 0), 32), ((1, 1), (0, 1), 16)]:
        base = dict(alloc.live)
        alloc.arm(0)
        A = sp().sp_pack(coo.dims, coords, vals, lt, od, posBits=pb, crdBits=pb)
        # A fresh handle: the first call also builds the tables the handle caches (work partition,
        # widened copy of 16-bit storage), so those allocations are failure points too.  What a call
        # had cached before it failed stays with the handle (and is freed with it); its own scratch
        # must be back, which the comparison after sp_free below proves, a leak being owned by no one.
        for call in (lambda: sp().sp_spmm(A, Bd, out), lambda: sp().sp_spmv(A, xd, y)):
            for k in range(1, 50):
                alloc.arm(k)
                try:
                    call()
                except alloc.b.SpError as e:
                    assert e.code == SP_ERR_ALLOC and alloc.failed
                    continue
                assert not alloc.failed
                break
            else:
                raise AssertionError("the call never got through")
        alloc.arm(0)
        assert_close(sp().sp_spmm(A, Bd, out).cpu().numpy(), ref, bd, "after the failures")
        A.free()
        torch.cuda.synchronize()
        assert alloc.live == base, f"{lt} {od}: {len(alloc.live) - len(base)} allocation(s) outlive the handle"


def test_sddmm_mttkrp_spmspm_give_everything_back(alloc):
    s = I.config4(seed=7, n=512, nnz=4000)
    coords, vals = to_dev(s)
    A4, B4 = dev(I.dense_operand(7, 35, 512, 16)), dev(I.dense_operand(7, 36, 16, 512))
    alloc.arm(0)
    S = sp().sp_pack(s.dims, coords, vals, (0, 1))
    xv = torch.empty(S.nval, dtype=torch.float64, device="cuda")
    sp().sp_sddmm(S, A4, B4, xv)             # builds the handle's cached partition; what is left is per-call scratch
    assert sweep(alloc, lambda: sp().sp_sddmm(S, A4, B4, xv), cleanup=lambda r: None) >= 1
    t = I.config5(seed=7, dim=64, nnz=5000)
    tc, tv = to_dev(t)
    alloc.arm(0)
    T = sp().sp_pack(t.dims, tc, tv, (1, 1, 1))
    Bf, Cf = dev(I.dense_operand(7, 37, 64, 8)), dev(I.dense_operand(7, 38, 64, 8))
    M = torch.empty(64, 8, dtype=torch.float64, device="cuda")
    base = dict(alloc.live)
    for k in range(1, 20):                   # a fresh handle: the cached partition's three arrays are failure points
        alloc.arm(k)
        try:
            sp().sp_mttkrp(T, Bf, Cf, M)
        except alloc.b.SpError as e:
            assert e.code == SP_ERR_ALLOC
            torch.cuda.synchronize()
            assert alloc.live == base        # a partition is cached whole or not at all
            continue
        break
    assert k >= 4
    q = I.uniform_matrix(256, 256, 1500, seed=8)
    qc, qv = to_dev(q)
    alloc.arm(0)
    Q = sp().sp_pack(q.dims, qc, qv, (0, 1))
    assert sweep(alloc, lambda: sp().sp_spmspm(Q, Q)) >= 3
    S.free(); T.free(); Q.free()
