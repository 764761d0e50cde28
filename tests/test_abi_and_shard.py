"""CPU-side checks: the C-ABI library loads and exports what the header declares;
the column-slab partition (the multi-GPU path's host logic) reproduces the whole
vector, also as two gloo ranks."""
import ctypes
import os
import re
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import CSEROracle, grbs_mask
from paper_2007_13221_b200.shard import slab_of_rank

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    header = open(os.path.join(ROOT, "include", "cser.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(cser_[a-z0-9_]+)\s*\(", header))
    assert {"cser_create", "cser_step", "cser_read_state"} <= names and len(names) >= 12
    L = ctypes.CDLL(os.path.join(ROOT, "paper_2007_13221_b200", "libcser.so"))
    for nm in sorted(names):
        assert hasattr(L, nm), nm
    L.cser_last_error.restype = ctypes.c_char_p
    assert L.cser_last_error() == b""


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2007_13221_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libcser.so"))
    with pytest.raises(binding.CSERError):
        binding.lib()


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2007_13221_b200")
    for dp, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dp, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2007_13221_b200" not in src, f


@pytest.mark.parametrize("d,bs,world", [(1000, 16, 2), (1001, 16, 3), (35_748_708, 512, 8), (40, 256, 4)])
def test_slabs_tile_the_vector_in_whole_blocks(d, bs, world):
    prev_end, prev_b = 0, 0
    for r in range(world):
        c0, c1, b0 = slab_of_rank(d, bs, r, world)
        assert c0 == prev_end and b0 == prev_b and c0 == min(b0 * bs, d) and c1 >= c0
        prev_end, prev_b = c1, b0 + (c1 - c0 + bs - 1) // bs
    assert prev_end == d


def _problem():
    rng = np.random.default_rng(77)
    n, d, T = 4, 1000 + 8, 12
    x0 = rng.standard_normal(d).astype(np.float32)
    g = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(T)]
    return n, d, T, x0, g


class _SlabOracle(CSEROracle):
    """Oracle on a slab: same columns as a `cols` subset of the global vector."""


def _run_slab(rank, world):
    n, d, T, x0, g = _problem()
    bs = 16
    c0, c1, b0 = slab_of_rank(d, bs, rank, world)
    o = CSEROracle(d, n, bs, 4, 2, 3, 0.1, 0.9, 5, dtype=np.float32, cols=np.arange(c0, c1))
    o.set_x0(x0[c0:c1])
    for gt in g:
        o.step(gt[:, c0:c1])
    return c0, c1, o


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    c0, c1, o = _run_slab(rank, world)
    n, d = o.n, o.d
    full = torch.zeros((2, n, d))
    full[0, :, c0:c1] = torch.from_numpy(o.x)
    full[1, :, c0:c1] = torch.from_numpy(o.e)
    dist.all_reduce(full)                      # only to assemble the result for checking
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)   # the bench's max-over-ranks timing reduction
    if rank == 0:
        q.put((full.numpy(), float(t)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_with_column_slabs_equal_the_single_process_result():
    n, d, T, x0, g = _problem()
    whole = CSEROracle(d, n, 16, 4, 2, 3, 0.1, 0.9, 5, dtype=np.float32)
    whole.set_x0(x0)
    for gt in g:
        whole.step(gt)
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    [p.start() for p in procs]
    full, tmax = q.get(timeout=120)
    [p.join(60) for p in procs]
    assert all(p.exitcode == 0 for p in procs)
    assert np.array_equal(full[0], whole.x) and np.array_equal(full[1], whole.e)
    assert tmax == 2.0
    # the slab's mask is the slab of the global mask
    c0, c1, b0 = slab_of_rank(d, 16, 1, 2)
    B = (d + 15) // 16
    assert np.array_equal(grbs_mask(5, 3, 0, B - b0, 4, block_begin=b0), grbs_mask(5, 3, 0, B, 4)[b0:])
