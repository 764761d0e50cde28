"""The allocation-free entry point against the handle-based one.

Some callers cannot call cudaMalloc where they step the optimizer (all device memory
belongs to their framework's pool, or an allocation would stall their other streams).
cser_step_noalloc serves them: the caller owns x, e, m and the step counter, and the
masks live in a fixed array inside the library.  This file is named so that pytest
collects it last; it must pass alone in a fresh process and after all other tests.
"""
import numpy as np
import pytest
import torch

from oracle import CSEROracle
from paper_2007_13221_b200 import binding as b, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("beta,d", [(0.9, 200_000 + 36), (0.0, 50_001)])
def test_noalloc_step_equals_handle_step_on_consecutive_calls(beta, d):
    import __graft_entry__
    __graft_entry__.build()
    torch.cuda.set_device(0)
    w = synth.CONFIGS[2].scaled(d=d, steps=6)
    n, bs, R1, R2, H, eta, seed = w.n_workers, w.block_size, 4, 2, 2, w.eta, 11
    ref = b.CSER(d, n, bs, R1, R2, H, eta, beta, seed)
    x0 = synth.x0(w, DEV)
    ref.set_x0(x0)
    x = x0[None, :].repeat(n, 1).contiguous()
    e = torch.zeros_like(x)
    m = torch.zeros_like(x) if beta else None
    for t in range(1, w.steps + 1):                # t = 2, 4, 6 are reset steps
        g = synth.gradients(w, t, DEV)
        ref.step(g)
        b.cser_step_noalloc(d, n, bs, R1, R2, H, eta, beta, seed, t, g, x, e, m)
        torch.cuda.synchronize()
        # same tolerance as the other GPU tests use between identical arithmetic: exact
        assert torch.equal(ref.state(b.STATE_X), x), t
        assert torch.equal(ref.state(b.STATE_E), e), t
        if beta:
            assert torch.equal(ref.state(b.STATE_M), m), t
    ref.close()


def test_noalloc_step_equals_the_float32_oracle():
    """Directly against the CPU oracle (float32 evaluation, same operation order: equal bits), not only
    against the handle-based entry point."""
    torch.cuda.set_device(0)
    d, n, bs, R1, R2, H, eta, beta, seed = 30_000 + 12, 5, 128, 3, 2, 2, 0.1, 0.9, 21
    rng = np.random.default_rng(7)
    x0 = rng.standard_normal(d).astype(np.float32)
    ref = CSEROracle(d, n, bs, R1, R2, H, eta, beta, seed, dtype=np.float32)
    ref.set_x0(x0)
    x = torch.from_numpy(np.tile(x0, (n, 1))).to(DEV)
    e, m = torch.zeros_like(x), torch.zeros_like(x)
    for t in range(1, 8):
        g = rng.standard_normal((n, d)).astype(np.float32)
        ref.step(g)
        b.cser_step_noalloc(d, n, bs, R1, R2, H, eta, beta, seed, t, torch.from_numpy(g).to(DEV), x, e, m)
        torch.cuda.synchronize()
        for got, want, name in ((x, ref.x, "x"), (e, ref.e, "e"), (m, ref.m, "m")):
            assert np.array_equal(got.cpu().numpy(), want), (t, name)


def test_noalloc_at_its_largest_vector_on_a_side_stream_allocates_nothing():
    """Exactly CSER_NOALLOC_MAX_BLOCKS blocks, every block selected (R1 = 1), so the list fills the
    scratch to its last entry, right below the three counters; three or more consecutive steps on a side
    stream, so that every counter takes its turn; and the free device memory does not move."""
    torch.cuda.set_device(0)
    max_blocks, bs, n = 262144, 4, 1
    d = max_blocks * bs
    R1, R2, H, eta, beta, seed = 1, 2, 1, 0.1, 0.0, 3
    ref = b.CSER(d, n, bs, R1, R2, H, eta, beta, seed)
    x0 = torch.randn(d, device=DEV)
    ref.set_x0(x0)
    x = x0[None, :].clone()
    e = torch.zeros_like(x)
    grads = [torch.randn((n, d), device=DEV) for _ in range(5)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b.cser_step_noalloc(d, n, bs, R1, R2, H, eta, beta, seed, 1, grads[0], x, e, None)   # warm-up call
        side.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        for t in range(2, 6):
            b.cser_step_noalloc(d, n, bs, R1, R2, H, eta, beta, seed, t, grads[t - 1], x, e, None)
        side.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
    for t in range(1, 6):
        ref.step(grads[t - 1])
    torch.cuda.synchronize()
    assert torch.equal(ref.state(b.STATE_X), x)
    assert torch.equal(ref.state(b.STATE_E), e)
    ref.close()


def test_noalloc_rejects_vectors_beyond_its_built_in_scratch():
    torch.cuda.set_device(0)
    L = b.lib()
    max_blocks = 262144
    z = torch.zeros(8, device=DEV)
    rc = L.cser_step_noalloc((max_blocks + 1) * 4, 1, 4, 2, 2, 2, 0.1, 0.0, 0, 1,
                             z.data_ptr(), z.data_ptr(), z.data_ptr(), None, None)
    assert rc == -1 and "exceed" in b.cser_last_error()
    rc = L.cser_step_noalloc(8, 1, 4, 2, 2, 2, 0.1, 0.0, 0, 0, z.data_ptr(), z.data_ptr(), z.data_ptr(), None, None)
    assert rc == -1                                 # t is 1-based


@pytest.mark.parametrize("d,n,bs,beta", [(10_000 + 36, 8, 256, 0.9), (1001, 3, 7, 0.9), (4099, 5, 64, 0.0),
                                         (70_000, 16, 1024, 0.9)])
def test_kernels_never_write_outside_the_arrays_they_are_given(d, n, bs, beta):
    """Guard bands: with the caller-owned arrays of the allocation-free entry point, x, e, m and the
    gradients sit inside larger buffers filled with a sentinel; after steps through every kernel path
    (plain and reset steps, selected and unselected blocks, ragged last block) the sentinels around
    each array must be untouched."""
    torch.cuda.set_device(0)
    pad, sentinel = 4096, 12345.0
    total = n * d

    def guarded():
        buf = torch.full((total + 2 * pad,), sentinel, dtype=torch.float32, device=DEV)
        return buf, buf[pad:pad + total].view(n, d)

    (bx, x), (be, e), (bm, m), (bg, g) = guarded(), guarded(), guarded(), guarded()
    x.copy_(torch.randn(d, device=DEV)[None, :].expand(n, d))
    e.zero_(), m.zero_()
    for t in range(1, 9):                                   # H = 2: four reset steps
        g.copy_(torch.randn((n, d), device=DEV))
        b.cser_step_noalloc(d, n, bs, 2, 2, 2, 0.1, beta, 5, t, g, x, e, m if beta else None)
    torch.cuda.synchronize()
    for name, buf in (("x", bx), ("e", be), ("m", bm), ("g", bg)):
        assert bool((buf[:pad] == sentinel).all()) and bool((buf[pad + total:] == sentinel).all()), name
    assert bool(torch.isfinite(x).all()) and bool((x != sentinel).any())
    if not beta:
        assert bool((m == 0).all())                         # no momentum: m is never touched
