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

from oracle import CSEROracle, exact_count, get_p, grbs_mask, grbs_mask_exact
from paper_2007_13221_b200.shard import slab_of_rank, workers_of_rank

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


def test_header_is_plain_c_and_the_library_links_from_c(tmp_path):
    import subprocess
    import __graft_entry__
    __graft_entry__.build()
    pkg = os.path.join(ROOT, "paper_2007_13221_b200")
    exe = str(tmp_path / "abi_c_check")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "abi_c_check.c"), "-o", exe, "-L", pkg, "-l:libcser.so",
           "-Wl,-rpath," + pkg]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    run = subprocess.run([exe], capture_output=True, text=True)
    assert run.returncode == 0, (run.returncode, run.stdout, run.stderr)
    # every function the header declares is exercised by the C program
    header = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "cser.h")).read(), flags=re.S)
    declared = set(re.findall(r"\b(cser_[a-z0-9_]+)\s*\(", header))
    used = set(re.findall(r"\b(cser_[a-z0-9_]+)\b", open(os.path.join(ROOT, "tests", "abi_c_check.c")).read()))
    assert declared <= used, declared - used


def test_built_library_is_stamped_with_the_id_of_its_sources():
    """build() stamps libcser.so with an id over its sources and flags and rebuilds when they differ, so a
    stale binary cannot pass for a current one."""
    import __graft_entry__
    __graft_entry__.build()
    from paper_2007_13221_b200 import binding
    rec = __graft_entry__.library_record()
    assert rec["matches_sources"] and len(rec["build_id"]) == 16, rec
    assert binding.cser_build_id() == __graft_entry__.source_id(
        os.path.join(ROOT, "paper_2007_13221_b200", "csrc", "cser.cu"))


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


# ---------------------------------------------------------------- worker-sharded decomposition over gloo
def _wshard_worker(rank, world, port, q):
    """Each rank holds some workers, sums its own selected-block values, all-reduces the packed
    message and applies the mean - the host-side algebra of the worker-sharded step, in NumPy."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n, d, T, x0, g = _problem()
    bs, R1, R2, H, eta, beta, seed = 16, 4, 2, 3, np.float64(np.float32(0.1)), np.float64(np.float32(0.9)), 5
    B = (d + bs - 1) // bs
    first, cnt = workers_of_rank(n, rank, world)
    x = np.repeat(x0.astype(np.float64)[None, :], cnt, 0)
    e, m = np.zeros_like(x), np.zeros_like(x)
    blk = np.arange(d) // bs
    for t, gt in enumerate(g, 1):
        is_reset = t % H == 0
        sg = grbs_mask_exact(seed, t, 0, B, R1)[blk] != 0
        sr = (grbs_mask_exact(seed, t, 1, B, R2)[blk] != 0) if is_reset else np.zeros(d, bool)
        p, m = get_p(m, gt[first:first + cnt].astype(np.float64), eta, beta)
        x_half = np.where(sg[None, :], x, x - p)                    # selected: wait for the mean
        e_half = np.where(sg[None, :], e, e - p)
        msg = torch.from_numpy(np.concatenate([p[:, sg].sum(0), e_half[:, sr].sum(0)]))
        assert msg.numel() == int(sg.sum()) + int(sr.sum())
        dist.all_reduce(msg)
        msg = msg.numpy() / n
        x_half[:, sg] -= msg[: int(sg.sum())][None, :]
        if is_reset:
            x_half[:, sr] = (x_half[:, sr] - e_half[:, sr]) + msg[int(sg.sum()):][None, :]
            e_half[:, sr] = 0
        x, e = x_half, e_half
    out = torch.zeros((2, n, d), dtype=torch.float64)
    out[0, first:first + cnt] = torch.from_numpy(x)
    out[1, first:first + cnt] = torch.from_numpy(e)
    dist.all_reduce(out)
    if rank == 0:
        q.put(out.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_worker_sharded_decomposition_over_two_gloo_ranks_matches_the_oracle():
    n, d, T, x0, g = _problem()
    ref = CSEROracle(d, n, 16, 4, 2, 3, 0.1, 0.9, 5, dtype=np.float64, exact_count=True)
    ref.set_x0(x0)
    for gt in g:
        ref.step(gt)
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_wshard_worker, args=(r, 2, port, q)) for r in range(2)]
    [p.start() for p in procs]
    out = q.get(timeout=120)
    [p.join(60) for p in procs]
    assert all(p.exitcode == 0 for p in procs)
    assert np.allclose(out[0], ref.x, rtol=1e-12, atol=1e-12) and np.allclose(out[1], ref.e, rtol=1e-12, atol=1e-12)
    assert [workers_of_rank(8, r, 3) for r in range(3)] == [(0, 3), (3, 3), (6, 2)]
