"""Host-side logic of bench.py that runs on more than one rank, on CPU with gloo (world size 2),
and the arithmetic of the work model."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    assert bench.dist_env() == (rank, rank, world)
    bench.dist_barrier()
    slow = bench.dist_max(10.0 + 5.0 * rank, "cpu")        # the slowest rank's time is what counts
    out.put((rank, slow))
    dist.destroy_process_group()


def test_max_over_ranks_with_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0), (1, 15.0)]


def test_single_process_identity():
    import bench
    assert bench.dist_max(3.5, "cpu") == 3.5
    bench.dist_barrier()


def test_work_model_counts():
    import bench
    wl = bench.make_workload(small=True, seed=0)
    m = bench.work_model(wl)
    c3, c5 = wl["c3"], wl["c5"]
    assert m["spmm_csc"]["flops"] == 2 * 32 * c3.nnz
    assert m["spmv_csr"]["flops"] == 2 * wl["c1b"].nnz
    assert m["sddmm_csr"]["flops"] == wl["c4"].nnz * 257
    assert m["mttkrp_csf"]["flops"] == 2 * 32 * (c5.nnz + wl["F5"])
    # compulsory bytes: 12 B per stored entry (4 B coordinate + 8 B value) plus each dense operand once
    assert m["spmm_csc"]["bytes"] == 12 * c3.nnz + 4 * (c3.dims[1] + 1) + 8 * 32 * sum(c3.dims)
    assert all(v["bytes"] > 0 for v in m.values())
