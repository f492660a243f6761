"""The bounds-checking build (libsp_debug_bounds.so, -DSP_DEBUG_BOUNDS): every index a kernel derives
from stored positions or coordinates is checked on the device; a bad one is recorded and replaced by
a valid one, and the call returns SP_ERR_OUT_OF_RANGE - never a trap or a fault.  It stands in for a
memory checker on machines where none may be run.

The build is selected per process (SP_DEBUG_BOUNDS=1), so the checks run in a child process:
  1. small parity cases of the four kernels give the oracle's results with no status raised;
  2. a coordinate overwritten with an out-of-range value makes the call report status 3, after which
     the handle, repaired, works again.  The operand that the bad coordinate indexes is allocated
     twice as long as declared, so the address would be inside the allocation even without the check."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np
import torch
import oracle as O
import paper_2202_04305_b200.binding as sp
from paper_2202_04305_b200 import inputs as I
from gpu_util import MATRIX_ENCODINGS, assert_close, dev, to_dev

assert sp.DEBUG_BOUNDS and sp._LIB_PATH.endswith("libsp_debug_bounds.so")

# 1. parity through the checking build
coo = I.config2(seed=3, n=700)
coords, vals = to_dev(coo)
B = I.dense_operand(3, 31, 700, 12)
x = I.uniform_pm1(3, 32, 700)
Cref, Cb = O.spmm(700, coo.coords[0], coo.coords[1], coo.vals, B)
yref, yb = O.spmv(700, coo.coords[0], coo.coords[1], coo.vals, x)
for enc, (lt, od) in MATRIX_ENCODINGS.items():
    A = sp.sp_pack(coo.dims, coords, vals, lt, od)
    assert_close(sp.sp_spmm(A, dev(B)).cpu().numpy(), Cref, Cb, enc)
    assert_close(sp.sp_spmv(A, dev(x)).cpu().numpy(), yref, yb, enc)
band = I.row_band_matrix(400, 5, seed=4)                 # long rows: the merge-path SpMV
bc, bv = to_dev(band)
xb = I.uniform_pm1(4, 1, 400)
r, b = O.spmv(400, band.coords[0], band.coords[1], band.vals, xb)
assert_close(sp.sp_spmv(sp.sp_pack(band.dims, bc, bv, (0, 1)), dev(xb)).cpu().numpy(), r, b, "band")
s = I.config4(seed=3, n=512, nnz=4000)
S = sp.sp_pack(s.dims, *to_dev(s), (0, 1))
A4, B4 = I.dense_operand(3, 35, 512, 24), I.dense_operand(3, 36, 24, 512)
xe, xbd = O.sddmm(s.coords[0], s.coords[1], s.vals, A4, B4)
ep = O.pack(s.dims, s.coords, s.vals, (0, 1)).entry_pos
got = sp.sp_sddmm(S, dev(A4), dev(B4)).cpu().numpy()
assert_close(got[ep], xe, xbd, "sddmm")
t = I.config5(seed=3, dim=96, nnz=20000)
tc, tv = to_dev(t)
Bf, Cf = I.dense_operand(3, 37, 96, 8), I.dense_operand(3, 38, 96, 8)
Mref, Mb = O.mttkrp(96, *t.coords, t.vals, Bf, Cf)
for lt in [(1, 1, 1), (0, 1, 1)]:
    T = sp.sp_pack(t.dims, tc, tv, lt)
    assert_close(sp.sp_mttkrp(T, dev(Bf), dev(Cf)).cpu().numpy(), Mref, Mb, f"mttkrp {lt}")

# dense inner level (both feeds of the SpMM, SpMV, SDDMM) and the all-sparse product
small = I.uniform_matrix(300, 260, 9000, seed=5)
sc, sv = to_dev(small)
Bs, xs = I.dense_operand(5, 31, 260, 12), I.uniform_pm1(5, 32, 260)
Cs, Csb = O.spmm(300, small.coords[0], small.coords[1], small.vals, Bs)
ys, ysb = O.spmv(300, small.coords[0], small.coords[1], small.vals, xs)
for lt, od in [((1, 0), (0, 1)), ((0, 0), (0, 1)), ((1, 0), (1, 0))]:
    A = sp.sp_pack(small.dims, sc, sv, lt, od)
    assert_close(sp.sp_spmm(A, dev(Bs)).cpu().numpy(), Cs, Csb, f"dense inner {lt} {od}")
    assert_close(sp.sp_spmm(A, dev(Bs[:, :7].copy())).cpu().numpy(), Cs[:, :7], Csb[:, :7], "dense inner, odd width")
    assert_close(sp.sp_spmv(A, dev(xs)).cpu().numpy(), ys, ysb, f"dense inner spmv {lt} {od}")
P, Q = I.uniform_matrix(120, 90, 900, seed=6), I.uniform_matrix(90, 150, 1100, seed=7)
hP, hQ = sp.sp_pack(P.dims, *to_dev(P), (0, 1)), sp.sp_pack(Q.dims, *to_dev(Q), (0, 1))
hC = sp.sp_spmspm(hP, hQ)
pos, crdC, valC, bdC = O.spmspm(120, 90, 150, P.coords[0], P.coords[1], P.vals, Q.coords[0], Q.coords[1], Q.vals)
assert np.array_equal(hC.coordinates(1).cpu().numpy().astype(np.int64), crdC)
assert_close(hC.values().cpu().numpy(), valC, bdC, "spmspm")

# 2. a coordinate out of range: status 3, no fault; operands hold twice the declared rows
n = 700
A = sp.sp_pack(coo.dims, coords, vals, (0, 1))
crd = A.coordinates(1)                     # a writable view of the handle's own array
x2 = torch.zeros(2 * n, dtype=torch.float64, device="cuda"); x2[:n] = dev(x)
B2 = torch.zeros(2 * n, 12, dtype=torch.float64, device="cuda"); B2[:n] = dev(B)
keep = int(crd[7])
crd[7] = n + 3
for call in (lambda: sp.sp_spmv(A, x2[:n]), lambda: sp.sp_spmm(A, B2[:n])):
    try:
        call()
    except sp.SpError as e:
        assert e.code == 3, e.code
    else:
        raise AssertionError("the bad coordinate went unnoticed")
crd[7] = keep
assert_close(sp.sp_spmv(A, x2[:n]).cpu().numpy(), yref, yb, "after repair")
assert_close(sp.sp_spmm(A, B2[:n]).cpu().numpy(), Cref, Cb, "after repair")

Ad = sp.sp_pack(small.dims, sc, sv, (1, 0), (0, 1))          # CDR: the stored row numbers address the output
c0 = Ad.coordinates(0)
keep = int(c0[3])
c0[3] = 300 + 2
Cbig = torch.zeros(2 * 300, 12, dtype=torch.float64, device="cuda")
ybig = torch.zeros(2 * 300, dtype=torch.float64, device="cuda")
for call in (lambda: sp.sp_spmm(Ad, dev(Bs), Cbig[:300]), lambda: sp.sp_spmv(Ad, dev(xs), ybig[:300])):
    try:
        call()
    except sp.SpError as e:
        assert e.code == 3, e.code
    else:
        raise AssertionError("the bad row number went unnoticed")
c0[3] = keep
assert_close(sp.sp_spmm(Ad, dev(Bs), Cbig[:300]).cpu().numpy(), Cs, Csb, "dense inner after repair")

T = sp.sp_pack(t.dims, tc, tv, (1, 1, 1))
C2 = torch.zeros(2 * 96, 8, dtype=torch.float64, device="cuda"); C2[:96] = dev(Cf)
k = T.coordinates(2)
keep = int(k[11])
k[11] = 96 + 5
try:
    sp.sp_mttkrp(T, dev(Bf), C2[:96])
except sp.SpError as e:
    assert e.code == 3, e.code
else:
    raise AssertionError("the bad leaf coordinate went unnoticed")
k[11] = keep
assert_close(sp.sp_mttkrp(T, dev(Bf), C2[:96]).cpu().numpy(), Mref, Mb, "mttkrp after repair")
torch.cuda.synchronize()
print("debug bounds ok")
'''


def test_checking_build_in_a_child_process():
    from paper_2202_04305_b200 import build
    build.build(debug_bounds=True)
    env = dict(os.environ, SP_DEBUG_BOUNDS="1", PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests")]))
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "debug bounds ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
