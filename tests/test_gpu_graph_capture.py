"""The compute calls inside a CUDA graph: after one eager call (which builds the handle's cached work
partition) sp_spmv / sp_spmm / sp_sddmm / sp_mttkrp only enqueue stream-ordered work and take their
scratch from the installed (caching) allocator, so a captured graph replays them on new operand values."""
import numpy as np
import pytest

from paper_2202_04305_b200 import inputs as I
from gpu_util import sp, to_dev, dev, assert_close

pytestmark = pytest.mark.gpu


def _replay_and_check(make_call, out, operands, new_values, check):
    import torch
    make_call()                                   # eager: builds whatever the handle caches
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        make_call()                               # allocator warm-up on the capture stream
        side.synchronize()
        with torch.cuda.graph(g, stream=side):
            make_call()
    for vals in new_values:                       # new operand values in the same buffers
        for buf, v in zip(operands, vals):
            buf.copy_(torch.as_tensor(v, device="cuda"))
        out.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        check(out.cpu().numpy(), vals)


@pytest.mark.parametrize("lt,od", [((0, 1), (0, 1)), ((1, 1), (0, 1)), ((0, 1), (1, 0)), ((1, 0), (0, 1))])
def test_spmv_and_spmm_replay(oracle, lt, od):
    import torch
    b = sp()
    coo = I.uniform_matrix(700, 650, 20000, seed=3)
    A = b.sp_pack(coo.dims, *to_dev(coo), lt, od)
    x = dev(I.uniform_pm1(1, 1, 650)); y = torch.empty(700, dtype=torch.float64, device="cuda")
    news = [(I.uniform_pm1(1, s, 650),) for s in (2, 3)]

    def check_v(got, vals):
        ref, bd = oracle.spmv(700, coo.coords[0], coo.coords[1], coo.vals, vals[0])
        assert_close(got, ref, bd, "captured spmv")
    _replay_and_check(lambda: b.sp_spmv(A, x, y), y, [x], news, check_v)

    B = dev(I.dense_operand(2, 1, 650, 16)); Cm = torch.empty((700, 16), dtype=torch.float64, device="cuda")
    newm = [(I.dense_operand(2, s, 650, 16),) for s in (2, 3)]

    def check_m(got, vals):
        ref, bd = oracle.spmm(700, coo.coords[0], coo.coords[1], coo.vals, vals[0])
        assert_close(got, ref, bd, "captured spmm")
    _replay_and_check(lambda: b.sp_spmm(A, B, Cm), Cm, [B], newm, check_m)


def test_sddmm_and_mttkrp_replay(oracle):
    import torch
    b = sp()
    coo = I.uniform_matrix(300, 280, 6000, seed=5)
    S = b.sp_pack(coo.dims, *to_dev(coo), (1, 1))
    ep = oracle.pack(coo.dims, coo.coords, coo.vals, (1, 1)).entry_pos
    A = dev(I.dense_operand(3, 1, 300, 64)); B = dev(I.dense_operand(3, 2, 64, 280))
    xv = torch.empty(S.nval, dtype=torch.float64, device="cuda")
    news = [(I.dense_operand(3, s, 300, 64), I.dense_operand(3, s + 10, 64, 280)) for s in (3, 4)]

    def check_s(got, vals):
        xe, be = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, vals[0], vals[1])
        ref = np.empty_like(xe); bd = np.empty_like(be)
        ref[ep] = xe; bd[ep] = be
        assert_close(got, ref, bd, "captured sddmm")
    _replay_and_check(lambda: b.sp_sddmm(S, A, B, xv), xv, [A, B], news, check_s)

    t3 = I.uniform_tensor((60, 50, 40), 9000, seed=6)
    T = b.sp_pack(t3.dims, *to_dev(t3), (1, 1, 1))
    Bf = dev(I.dense_operand(4, 1, 50, 32)); Cf = dev(I.dense_operand(4, 2, 40, 32))
    M = torch.empty((60, 32), dtype=torch.float64, device="cuda")
    newf = [(I.dense_operand(4, s, 50, 32), I.dense_operand(4, s + 10, 40, 32)) for s in (3, 4)]

    def check_t(got, vals):
        ref, bd = oracle.mttkrp(60, t3.coords[0], t3.coords[1], t3.coords[2], t3.vals, vals[0], vals[1])
        assert_close(got, ref, bd, "captured mttkrp")
    _replay_and_check(lambda: b.sp_mttkrp(T, Bf, Cf, M), M, [Bf, Cf], newf, check_t)
