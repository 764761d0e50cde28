"""Worker-sharded step (each rank holds some of the workers; one all-reduce per step).

On one GPU the ranks are emulated one after the other: every rank packs, the messages are
added (standing in for the all-reduce), every rank applies.  No kernel waits on another.
"""
import os
import socket

import numpy as np
import pytest
import torch

from oracle import CSEROracle, exact_count
from paper_2007_13221_b200 import binding as b
from paper_2007_13221_b200.shard import workers_of_rank

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__
    __graft_entry__.build()
    torch.cuda.set_device(0)


def _problem(d, n, steps, seed=0):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d).astype(np.float32)
    g = [(rng.standard_normal(d)[None, :] + 0.5 * rng.standard_normal((n, d))).astype(np.float32)
         for _ in range(steps)]
    return x0, g


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", [(4096 + 40, 8, 256, 4, 2, 3, 0.9), (1001, 3, 7, 2, 3, 2, 0.9),
                                                 (20_000, 16, 1024, 2, 2, 1, 0.0)])
def test_one_rank_holding_all_workers_equals_the_single_gpu_step_exactly(d, n, bs, R1, R2, H, beta):
    x0, g = _problem(d, n, 9)
    a = b.CSER(d, n, bs, R1, R2, H, 0.1, beta, 5, flags=b.FLAG_EXACT_COUNT)
    c = b.WorkerShardedCSER(d, n, n, bs, R1, R2, H, 0.1, beta, 5)
    a.set_x0(torch.from_numpy(x0).to(DEV)), c.set_x0(torch.from_numpy(x0).to(DEV))
    for t, gt in enumerate(g, 1):
        gd = torch.from_numpy(gt).to(DEV)
        a.step(gd)
        assert c.message_elems() == (exact_count(a.B, R1) + (exact_count(a.B, R2) if t % H == 0 else 0)) * bs
        c.step(gd)
        for which in (b.STATE_MASK_G, b.STATE_X, b.STATE_E) + ((b.STATE_M,) if beta else ()):
            assert torch.equal(a.state(which), c.state(which)), (t, which)
    a.close(), c.close()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", [(4096 + 40, 8, 256, 4, 2, 3, 0.9), (1001, 5, 7, 2, 3, 2, 0.0),
                                                 (50_000, 16, 512, 8, 4, 4, 0.9)])
def test_emulated_ranks_match_the_oracle(world, d, n, bs, R1, R2, H, beta):
    steps = 24
    x0, g = _problem(d, n, steps, seed=world)
    ref32 = CSEROracle(d, n, bs, R1, R2, H, 0.1, beta, 9, dtype=np.float32, exact_count=True)
    ref64 = CSEROracle(d, n, bs, R1, R2, H, 0.1, beta, 9, dtype=np.float64, exact_count=True)
    ref32.set_x0(x0), ref64.set_x0(x0)
    ranks = []
    for r in range(world):
        first, cnt = workers_of_rank(n, r, world)
        h = b.WorkerShardedCSER(d, cnt, n, bs, R1, R2, H, 0.1, beta, 9)
        h.set_x0(torch.from_numpy(x0).to(DEV))
        ranks.append((first, cnt, h))
    for t, gt in enumerate(g, 1):
        ref32.step(gt), ref64.step(gt)
        msgs = [h.pack(torch.from_numpy(np.ascontiguousarray(gt[first:first + cnt])).to(DEV))
                for first, cnt, h in ranks]
        total = torch.stack([m.clone() for m in msgs]).sum(0)          # the all-reduce
        for (_, _, h), m in zip(ranks, msgs):
            m.copy_(total)
            h.apply()
        if t in (1, steps):
            for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
                got = torch.cat([h.state(which) for _, _, h in ranks]).cpu().numpy()
                w64, w32 = getattr(ref64, name), getattr(ref32, name)
                if t == 1:
                    assert (np.abs(got - w64) <= 1e-6 * np.abs(w64) + 1e-7).all(), name
                rms = float(np.sqrt((w64**2).mean()))
                assert (np.abs(got - w64) <= 1e-4 * np.abs(w64) + 1e-4 * rms).all(), name
                assert np.abs(got - w32).max() <= 1e-5 * max(1.0, np.abs(w32).max()), name
        assert np.array_equal(ranks[0][2].state(b.STATE_MASK_G).cpu().numpy(), ref32.mask_g)
    [h.close() for _, _, h in ranks]


def test_step_through_a_real_nccl_group_of_one():
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device(DEV))
    try:
        d, n, bs = 10_000, 4, 64
        x0, g = _problem(d, n, 6)
        a = b.CSER(d, n, bs, 4, 2, 2, 0.1, 0.9, 1, flags=b.FLAG_EXACT_COUNT)
        c = b.WorkerShardedCSER(d, n, n, bs, 4, 2, 2, 0.1, 0.9, 1)
        a.set_x0(torch.from_numpy(x0).to(DEV)), c.set_x0(torch.from_numpy(x0).to(DEV))
        for gt in g:
            gd = torch.from_numpy(gt).to(DEV)
            a.step(gd)
            msg = c.pack(gd)
            dist.all_reduce(msg)                       # NCCL, one rank
            c.apply()
        assert torch.equal(a.state(b.STATE_X), c.state(b.STATE_X))
        a.close(), c.close()
    finally:
        dist.destroy_process_group()


def test_misuse_is_reported():
    L = b.lib()
    c = b.WorkerShardedCSER(1000, 2, 4, 10, 2, 2, 2, 0.1, 0.0, 0)
    g = torch.zeros((2, 1000), device=DEV)
    assert L.cser_step(c.h, g.data_ptr(), None) == -1                       # wrong entry point
    assert L.cser_wshard_apply(c.h, c.msg.data_ptr(), None) == -1            # nothing packed
    small = torch.zeros(4, device=DEV)
    assert L.cser_wshard_pack(c.h, g.data_ptr(), small.data_ptr(), 4, None) == -4
    c.pack(g)
    assert L.cser_wshard_pack(c.h, g.data_ptr(), c.msg.data_ptr(), c.msg.numel(), None) == -1   # apply pending
    c.apply()
    plain = b.CSER(1000, 2, 10, 2, 2, 2, 0.1, 0.0, 0)
    assert L.cser_wshard_message_elems(plain.h, 0) == -1
    assert not L.cser_create_wshard(1000, 5, 4, 10, 2, 2, 2, 0.1, 0.0, 0)    # n_local > n_total
    c.close(), plain.close()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two GPUs")
def test_two_ranks_on_two_gpus_with_an_nccl_all_reduce():
    """The workers split over two processes on two GPUs, the packed message summed by NCCL: every rank's state
    must match the oracle within the stated tolerances (the sum over workers is associated rank by rank)."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = {**os.environ, "NCCL_NVLS_ENABLE": "0"}
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port),
                          os.path.join(root, "tests", "wshard_ranks_check.py")],
                         capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0 and "WSHARD_RANKS_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]
