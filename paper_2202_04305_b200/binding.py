"""Thin ctypes binding over libsp.so: argument marshalling only.

Every function has the name and the meaning of the C entry point in
``include/sp.h``; torch supplies device memory and the current stream.
There is no fallback: if the library is missing, importing fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

DENSE, COMPRESSED = 0, 1
MAX_RANK = 5
DUP_SUM, DUP_ERROR = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
# SP_DEBUG_BOUNDS=1 in the environment selects the bounds-checking build of the same library (every
# index derived from stored positions / coordinates is checked on the device; a bad one makes the call
# return SP_ERR_OUT_OF_RANGE instead of reading or writing out of bounds).  Much slower; for debugging.
DEBUG_BOUNDS = os.environ.get("SP_DEBUG_BOUNDS", "") not in ("", "0")
_LIB_PATH = os.path.join(_HERE, "libsp_debug_bounds.so" if DEBUG_BOUNDS else "libsp.so")

SYMBOLS = ["sp_status_string", "sp_set_allocator", "sp_pack", "sp_free", "sp_info", "sp_positions",
           "sp_coordinates", "sp_values", "sp_unpack", "sp_spmv", "sp_spmm", "sp_sddmm", "sp_mttkrp",
           "sp_launch_count", "sp_spmv_static", "sp_mttkrp_mode", "sp_spmspm", "sp_convert", "sp_scale", "sp_vec_dot"]
SPMV_STATIC_MAX_ITEMS = 134217728


class SpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.sp_status_string(code).decode()} (status {code})")


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_2202_04305_b200.build"
                          f"{' --debug-bounds' if DEBUG_BOUNDS else ''}` (there is no CPU fallback)")
    lib = C.CDLL(_LIB_PATH)
    lib.sp_status_string.restype = C.c_char_p
    lib.sp_status_string.argtypes = [C.c_int]
    for name in SYMBOLS[1:]:
        getattr(lib, name).restype = C.c_int
    lib.sp_launch_count.restype = C.c_int64
    return lib


_lib = _load()

_ALLOC_T = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p)
_FREE_T = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p, C.c_void_p)


def _torch_alloc(nbytes, stream, ctx):
    try:
        return torch.cuda.caching_allocator_alloc(max(int(nbytes), 1), stream=int(stream or 0))
    except Exception:
        return None


def _torch_free(ptr, stream, ctx):
    if ptr:
        torch.cuda.caching_allocator_delete(ptr)


_alloc_cb = _ALLOC_T(_torch_alloc)
_free_cb = _FREE_T(_torch_free)
_allocator_set = False


def use_torch_allocator():
    """Route the library's allocations through torch's caching allocator."""
    global _allocator_set
    if not _allocator_set:
        _check(_lib.sp_set_allocator(_alloc_cb, _free_cb, None), "sp_set_allocator")
        _allocator_set = True


def _check(code, where):
    if code != 0:
        raise SpError(code, where)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dptr(t):
    return C.c_void_p(t.data_ptr() if t is not None and t.numel() else 0) if t is not None else C.c_void_p(0)


def _f64(t, name):
    if t.dtype != torch.float64 or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA float64 tensor")
    return t


class _DevArray:
    """Zero-copy view of library-owned device memory through __cuda_array_interface__."""

    def __init__(self, ptr, n, typestr, owner):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}
        self._owner = owner


_WIDTH_VIEW = {8: (torch.uint8, "|u1"), 16: (torch.uint16, "<u2"), 32: (torch.int32, "<i4"), 64: (torch.int64, "<i8")}


class SpTensor:
    """Owner of an sp_tensor handle."""

    def __init__(self, handle):
        self._h = handle
        rank = C.c_int()
        dims = (C.c_int64 * MAX_RANK)()
        lt = (C.c_int * MAX_RANK)()
        od = (C.c_int * MAX_RANK)()
        pb, cb = C.c_int(), C.c_int()
        _check(_lib.sp_info(self._h, C.byref(rank), dims, lt, od, C.byref(pb), C.byref(cb)), "sp_info")
        self.rank = rank.value
        self.dims = tuple(dims[i] for i in range(self.rank))
        self.lt = tuple(lt[i] for i in range(self.rank))
        self.ord = tuple(od[i] for i in range(self.rank))
        self.pos_bits, self.crd_bits = pb.value, cb.value

    def _arr(self, fn, level, bits):
        p, n = C.c_void_p(), C.c_int64()
        _check(fn(self._h, C.c_int(level), C.byref(p), C.byref(n)), fn.__name__)
        dt, typestr = _WIDTH_VIEW[bits]
        if n.value == 0 or not p.value:
            return torch.empty(0, dtype=dt, device="cuda")
        return torch.as_tensor(_DevArray(p.value, n.value, typestr, self), device="cuda")

    def positions(self, level):
        """pos[level] as a view of the device array (empty at dense levels): uint8 / uint16 for the
        narrow widths, a signed view of the unsigned words for 32 and 64 bits."""
        return self._arr(_lib.sp_positions, level, self.pos_bits)

    def coordinates(self, level):
        return self._arr(_lib.sp_coordinates, level, self.crd_bits)

    def values(self):
        p, n = C.c_void_p(), C.c_int64()
        _check(_lib.sp_values(self._h, C.byref(p), C.byref(n)), "sp_values")
        if n.value == 0:
            return torch.empty(0, dtype=torch.float64, device="cuda")
        return torch.as_tensor(_DevArray(p.value, n.value, "<f8", self), device="cuda")

    @property
    def nval(self):
        p, n = C.c_void_p(), C.c_int64()
        _check(_lib.sp_values(self._h, C.byref(p), C.byref(n)), "sp_values")
        return n.value

    def free(self):
        if self._h:
            _lib.sp_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def sp_pack(dims, coords, vals, dimLevelType, dimOrdering=None, posBits=32, crdBits=32, flags=DUP_SUM) -> SpTensor:
    """coords: one CUDA int32/int64 tensor per logical dimension; vals: CUDA float64."""
    use_torch_allocator()
    rank = len(dims)
    nnz = int(vals.numel())
    _f64(vals, "vals")
    bits = 64
    if rank and len(coords):
        bits = 32 if coords[0].dtype == torch.int32 else 64
    for c in coords:
        if not c.is_cuda or c.dtype not in (torch.int32, torch.int64) or (32 if c.dtype == torch.int32 else 64) != bits:
            raise TypeError("coords must be CUDA tensors of one integer type (int32 or int64)")
        if c.numel() != nnz or not c.is_contiguous():
            raise ValueError("each coords tensor must be contiguous with nnz entries")
    cptrs = (C.c_void_p * max(rank, 1))(*[c.data_ptr() if nnz else 0 for c in coords])
    h = C.c_void_p()
    lt = (C.c_int * rank)(*[int(t) for t in dimLevelType])
    od = (C.c_int * rank)(*[int(o) for o in dimOrdering]) if dimOrdering is not None else None
    _check(_lib.sp_pack(C.c_int(rank), (C.c_int64 * rank)(*[int(d) for d in dims]), C.c_int64(nnz), cptrs,
                        C.c_int(bits), _dptr(vals), lt, od, C.c_int(posBits), C.c_int(crdBits), C.c_uint(flags),
                        _stream(), C.byref(h)), "sp_pack")
    return SpTensor(h)


def sp_unpack(t: SpTensor):
    n = t.nval
    outs = [torch.empty(n, dtype=torch.int64, device="cuda") for _ in range(t.rank)]
    vals = torch.empty(n, dtype=torch.float64, device="cuda")
    cnt = C.c_int64()
    ptrs = (C.c_void_p * t.rank)(*[o.data_ptr() if n else 0 for o in outs])
    if n == 0:
        return outs, vals
    _check(_lib.sp_unpack(t._h, ptrs, _dptr(vals), C.byref(cnt), _stream()), "sp_unpack")
    return outs, vals


def sp_spmv(A: SpTensor, x, y=None):
    _f64(x, "x")
    if y is None:
        y = torch.empty(A.dims[0], dtype=torch.float64, device="cuda")
    _check(_lib.sp_spmv(A._h, _dptr(x), _dptr(y), _stream()), "sp_spmv")
    return y


def sp_spmv_static(A: SpTensor, x, y):
    """sp_spmv for callers that may not allocate: the library's scratch is a fixed device array.

    y must be supplied (this wrapper allocates nothing either).  Calls share that one array, so
    do not let two of them overlap on the GPU; see include/sp.h for the capacity and the rules."""
    _f64(x, "x"); _f64(y, "y")
    _check(_lib.sp_spmv_static(A._h, _dptr(x), _dptr(y), _stream()), "sp_spmv_static")
    return y


def sp_spmm(A: SpTensor, B, C_out=None):
    _f64(B, "B")
    N = B.shape[1]
    if C_out is None:
        C_out = torch.empty((A.dims[0], N), dtype=torch.float64, device="cuda")
    _check(_lib.sp_spmm(A._h, _dptr(B), C.c_int64(N), C.c_int64(B.stride(0)), _dptr(C_out), C.c_int64(C_out.stride(0)),
                        _stream()), "sp_spmm")
    return C_out


def sp_sddmm(S: SpTensor, A, B, x_vals=None):
    _f64(A, "A"); _f64(B, "B")
    if x_vals is None:
        x_vals = torch.empty(S.nval, dtype=torch.float64, device="cuda")
    _check(_lib.sp_sddmm(S._h, _dptr(A), C.c_int64(A.stride(0)), _dptr(B), C.c_int64(B.stride(0)),
                         C.c_int64(A.shape[1]), _dptr(x_vals), _stream()), "sp_sddmm")
    return x_vals


def sp_mttkrp(T: SpTensor, B, Cf, M=None):
    _f64(B, "B"); _f64(Cf, "C")
    if not (B.is_contiguous() and Cf.is_contiguous()):
        raise ValueError("factor matrices must be contiguous")
    R = B.shape[1]
    if M is None:
        M = torch.empty((T.dims[0], R), dtype=torch.float64, device="cuda")
    _check(_lib.sp_mttkrp(T._h, _dptr(B), _dptr(Cf), C.c_int64(R), _dptr(M), _stream()), "sp_mttkrp")
    return M


def sp_launch_count() -> int:
    return int(_lib.sp_launch_count())


def sp_mttkrp_mode(T: SpTensor, mode: int, factors, M=None):
    """factors: three CUDA float64 matrices (factors[mode] may be None); T stores dimension `mode` at level 0."""
    use = [f for d, f in enumerate(factors) if d != mode]
    for f in use:
        _f64(f, "factor")
        if not f.is_contiguous():
            raise ValueError("factor matrices must be contiguous")
    R = use[0].shape[1]
    if M is None:
        M = torch.empty((T.dims[mode], R), dtype=torch.float64, device="cuda")
    ptrs = (C.c_void_p * 3)(*[f.data_ptr() if (f is not None and d != mode) else 0 for d, f in enumerate(factors)])
    _check(_lib.sp_mttkrp_mode(T._h, C.c_int(mode), ptrs, C.c_int64(R), _dptr(M), _stream()), "sp_mttkrp_mode")
    return M


def sp_spmspm(A: SpTensor, B: SpTensor, posBits=32, crdBits=32) -> SpTensor:
    """C = A * B with A, B, C all CSR; returns a new handle."""
    use_torch_allocator()
    h = C.c_void_p()
    _check(_lib.sp_spmspm(A._h, B._h, C.c_int(posBits), C.c_int(crdBits), _stream(), C.byref(h)), "sp_spmspm")
    return SpTensor(h)


def sp_convert(t: SpTensor, dimLevelType, dimOrdering=None, posBits=32, crdBits=32) -> SpTensor:
    """Re-encode a tensor through coordinates (unpack + pack on the device)."""
    use_torch_allocator()
    h = C.c_void_p()
    lt = (C.c_int * t.rank)(*[int(x) for x in dimLevelType])
    od = (C.c_int * t.rank)(*[int(o) for o in dimOrdering]) if dimOrdering is not None else None
    _check(_lib.sp_convert(t._h, lt, od, C.c_int(posBits), C.c_int(crdBits), _stream(), C.byref(h)), "sp_convert")
    return SpTensor(h)


def sp_scale(x: SpTensor, c: float):
    _check(_lib.sp_scale(x._h, C.c_double(c), _stream()), "sp_scale")
    return x


def sp_vec_dot(a: SpTensor, b: SpTensor):
    out = torch.empty(1, dtype=torch.float64, device="cuda")
    _check(_lib.sp_vec_dot(a._h, b._h, _dptr(out), _stream()), "sp_vec_dot")
    return out
