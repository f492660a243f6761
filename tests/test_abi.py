"""Host-side checks that need no GPU: the library loads and exports what include/sp.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "sp.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2202_04305_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"sp_pack", "sp_spmv", "sp_spmm", "sp_sddmm", "sp_mttkrp", "sp_unpack", "sp_free"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    import paper_2202_04305_b200.binding as b
    assert sorted(b.SYMBOLS) == _declared()


def test_status_strings_without_a_device():
    import paper_2202_04305_b200.binding as b
    assert b._lib.sp_status_string(0) == b"ok"
    assert len({b._lib.sp_status_string(i) for i in range(9)}) == 9


def test_argument_errors_need_no_device():
    import paper_2202_04305_b200.binding as b
    h = ctypes.c_void_p()
    assert b._lib.sp_pack(0, None, 0, None, 32, None, None, None, 32, 32, 0, None, ctypes.byref(h)) == 1
    assert b._lib.sp_free(None) == 0
    assert b._lib.sp_spmv(None, None, None, None) == 1
    assert b._lib.sp_launch_count() >= 0
