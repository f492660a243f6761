"""Build libsp.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libsp.so")
SOURCES = ["api.cu", "pack.cu", "partition.cu", "spmv_spmm.cu", "sddmm.cu", "mttkrp.cu", "dense_inner.cu", "spmspm.cu", "vector_ops.cu"]
NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
# extra compiler flags, e.g. SP_NVCC_FLAGS="-DSP_SORT_MAX_BITS=8"; a change of them needs --force
NVCC_FLAGS += os.environ.get("SP_NVCC_FLAGS", "").split()


def _nvcc() -> str:
    for p in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if p and (os.path.sep not in p or os.path.exists(p)):
            return p
    return "nvcc"


def _newest_header() -> float:
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs.append(os.path.join(ROOT, "include", "sp.h"))
    return max(os.path.getmtime(h) for h in hs)


def _compile(src: str, verbose: bool, obj_dir: str = OBJ, extra=()) -> str:
    s = os.path.join(CSRC, src)
    o = os.path.join(obj_dir, src.replace(".cu", ".o"))
    if os.path.exists(o) and os.path.getmtime(o) >= max(os.path.getmtime(s), _newest_header()):
        return o
    cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode:
        raise RuntimeError(f"nvcc failed on {src}")
    return o


LIB_DEBUG = os.path.join(HERE, "libsp_debug_bounds.so")


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """debug_bounds: the checking build (-DSP_DEBUG_BOUNDS, see csrc/common.cuh) as a second library,
    libsp_debug_bounds.so, with its own object folder; the normal library is untouched."""
    obj_dir = OBJ + "_debug_bounds" if debug_bounds else OBJ
    lib = LIB_DEBUG if debug_bounds else LIB
    extra = ("-DSP_DEBUG_BOUNDS",) if debug_bounds else ()
    os.makedirs(obj_dir, exist_ok=True)
    if force:
        for f in os.listdir(obj_dir):
            os.remove(os.path.join(obj_dir, f))
    with cf.ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose, obj_dir, extra), SOURCES))
    if force or not os.path.exists(lib) or any(os.path.getmtime(o) > os.path.getmtime(lib) for o in objs):
        subprocess.check_call([_nvcc(), "-Wno-deprecated-gpu-targets", "-shared", "-o", lib] + objs + ["-lcudart"])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
