import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
LT = {"dense": 0, "compressed": 1}


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def load_golden(name):
    """Parse a tests/golden/*.txt fixture into a dict."""
    out = {"pos": {}, "crd": {}}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(":")
            rest = rest.strip()
            if key == "dims":
                out["dims"] = tuple(int(t) for t in rest.split())
            elif key == "lt":
                out["lt"] = tuple(LT[t] for t in rest.split())
            elif key == "ord":
                out["ord"] = tuple(int(t) for t in rest.split())
            elif key == "coo":
                ent = [[int(t) for t in e.split()] for e in rest.split(";")]
                out["coords"] = [np.array(c, dtype=np.int64) for c in zip(*ent)]
            elif key == "vals":
                out["vals"] = np.array([float(t) for t in rest.split()])
            elif key == "val":
                out["val"] = np.array([float(t) for t in rest.split()])
            elif key.startswith("pos"):
                out["pos"][int(key[3:])] = np.array([int(t) for t in rest.split()], dtype=np.int64)
            elif key.startswith("crd"):
                out["crd"][int(key[3:])] = np.array([int(t) for t in rest.split()], dtype=np.int64)
    return out


GOLDEN_FILES = sorted(f for f in os.listdir(GOLDEN) if f.endswith(".txt"))


def check_invariants(dims, lt, ord, pos, crd, val):
    """Storage invariants that hold for any input (Section 4.1's scheme)."""
    parents = 1
    for l, t in enumerate(lt):
        size = dims[ord[l]]
        if t == 0:
            assert pos[l] is None or len(pos[l]) == 0
            parents *= size
        else:
            p = np.asarray(pos[l]).astype(np.int64)
            c = np.asarray(crd[l]).astype(np.int64)
            assert p.size == parents + 1
            assert p[0] == 0 and p[-1] == c.size
            assert np.all(np.diff(p) >= 0)
            if c.size:
                assert c.min() >= 0 and c.max() < size
                inc = np.diff(c) > 0
                starts = p[1:-1]
                starts = starts[(starts > 0) & (starts < c.size)]
                ok = inc.copy()
                ok[starts - 1] = True      # a new segment may restart lower
                assert np.all(ok), "coordinates not strictly increasing inside a segment"
            parents = c.size
    assert np.asarray(val).size == parents


@pytest.fixture(scope="session")
def oracle():
    import oracle as O
    return O
