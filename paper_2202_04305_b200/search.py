"""Sparse state space search (Section 5.2): run one kernel over every storage encoding of the same
tensor, check that all results agree, and rank the encodings by time.

The paper's loop enumerates level types x dimension orderings x pointer widths x index widths and
calls verify(result) on each; this is the same loop over the encodings the library executes
(bit widths 8 to 64; a width the tensor overflows is skipped), with the agreement check between encodings taking the place of verify."""
from __future__ import annotations

import itertools
import statistics

import torch

from . import binding as sp

LEVELS_2D = [(sp.DENSE, sp.DENSE), (sp.DENSE, sp.COMPRESSED), (sp.COMPRESSED, sp.DENSE), (sp.COMPRESSED, sp.COMPRESSED)]
ORDERINGS_2D = [(0, 1), (1, 0)]
WIDTHS = [8, 16, 32, 64]


def _time(fn, reps):
    fn()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record(); b.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts)


def search_matrix_kernel(dims, coords, vals, kernel, levels=LEVELS_2D, orderings=ORDERINGS_2D, widths=WIDTHS, reps=5,
                         rtol=1e-9, max_dense_elems=1 << 26):
    """kernel(handle) -> CUDA tensor.  Returns a list of dicts (encoding, ms, max deviation from the
    first result), fastest first.  Encodings whose dense levels would not fit are skipped;
    raises AssertionError if two encodings disagree beyond rtol * max|result|."""
    first = None
    out = []
    for lt, od, pw, cw in itertools.product(levels, orderings, widths, widths):
        stored = 1
        for l in range(2):
            if lt[l] == sp.DENSE:
                stored *= dims[od[l]]
        if lt[1] == sp.DENSE and stored > max_dense_elems and lt[0] == sp.DENSE:
            continue
        if lt == (sp.COMPRESSED, sp.DENSE) and dims[od[1]] * min(dims[od[0]], int(vals.numel())) > max_dense_elems:
            continue
        try:
            h = sp.sp_pack(dims, coords, vals, lt, od, pw, cw)
            res = kernel(h)
        except sp.SpError as e:
            if e.code in (2, 4, 6):       # unsupported by this kernel, width overflow, allocation
                continue
            raise
        if first is None:
            first = res.clone()
        dev = float((res - first).abs().max()) if res.numel() else 0.0
        scale = float(first.abs().max()) if first.numel() else 0.0
        assert dev <= rtol * max(scale, 1e-300), f"encoding {lt} {od} {pw}/{cw} disagrees: {dev}"
        out.append({"levels": lt, "ordering": od, "posBits": pw, "crdBits": cw, "ms": _time(lambda: kernel(h), reps),
                    "max_dev": dev})
        h.free()
    return sorted(out, key=lambda r: r["ms"])
