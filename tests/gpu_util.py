"""Helpers shared by the GPU parity tests (kept import-safe on machines without CUDA)."""
import itertools

import numpy as np

TOL = 1e-12   # |gpu - oracle| <= TOL * sum|a*b| per output entry


def sp():
    import paper_2202_04305_b200.binding as b
    return b


def to_dev(coo, bits=32):
    import torch
    dt = torch.int32 if bits == 32 else torch.int64
    coords = [torch.as_tensor(np.ascontiguousarray(c), device="cuda").to(dt).contiguous() for c in coo.coords]
    vals = torch.as_tensor(coo.vals, device="cuda")
    return coords, vals


def dev(a):
    import torch
    return torch.as_tensor(np.ascontiguousarray(a), device="cuda")


def unsigned(t):
    """Overhead array of any width (8/16-bit unsigned, 32/64-bit words viewed as signed) as int64 values."""
    if t.numel() == 0:
        return np.empty(0, np.int64)
    a = t.cpu().numpy()
    return a.view({1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[a.dtype.itemsize]).astype(np.int64)


def assert_storage_equal(t, ref):
    """Bit-exact comparison of a packed handle with the oracle's storage."""
    for l in range(t.rank):
        p, c = unsigned(t.positions(l)), unsigned(t.coordinates(l))
        if ref.lt[l] == 1:
            assert np.array_equal(p, ref.pos[l]), f"pos[{l}] differs"
            assert np.array_equal(c, ref.crd[l]), f"crd[{l}] differs"
        else:
            assert p.size == 0 and c.size == 0
    v = t.values().cpu().numpy()
    assert v.size == ref.val.size
    assert np.array_equal(v.view(np.uint64), ref.val.view(np.uint64)), "values differ"


def assert_close(got, ref, bound, what=""):
    got = np.asarray(got); ref = np.asarray(ref); bound = np.asarray(bound)
    err = np.abs(got - ref)
    bad = err > TOL * bound
    assert not bad.any(), f"{what}: {int(bad.sum())} entries off, worst ratio {np.max(err / np.maximum(bound, 1e-300)):.3e}"
    assert np.all(got[bound == 0] == 0)


def all_encodings(rank):
    for lt in itertools.product((0, 1), repeat=rank):
        for od in itertools.permutations(range(rank)):
            yield lt, od


MATRIX_ENCODINGS = {"CSR": ((0, 1), (0, 1)), "DCSR": ((1, 1), (0, 1)), "CSC": ((0, 1), (1, 0)), "DCSC": ((1, 1), (1, 0))}
