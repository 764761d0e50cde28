"""Parity of the CUDA library (through its C ABI) with the CPU oracle.

Bars: GRBS masks bit-exact; float state within 1e-6 relative + 1e-7 absolute after
one step and 1e-4 relative (+ 1e-4 * RMS absolute, for entries that pass near zero)
after the full run, against the float64 oracle.  Because the kernel is compiled
without fused multiply-add and follows the same operation order, it must in addition
equal the float32 evaluation of the oracle exactly (signed zeros compare equal).
"""
import ctypes
import os

import numpy as np
import pytest
import torch

from _golden import read_hand_example
from oracle import CSEAOracle, CSERImpl2Oracle, CSEROracle, exact_count, grbs_mask, grbs_mask_exact, n_blocks, philox4x32_10, STREAM_GRAD, STREAM_RESET
from paper_2007_13221_b200 import binding as b, synth

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__
    __graft_entry__.build()
    torch.cuda.set_device(0)


@pytest.fixture(params=["one_launch_when_small", "three_kernels"])
def launch_path(request, monkeypatch):
    """Small problems (at most 256 MB moved per step) are stepped by one kernel that draws the masks itself; larger ones,
    and small ones created with CSER_FLAG_THREE_KERNELS, by the select / streaming / selected-block
    kernels.  A test that takes this fixture runs once on each path (same expected results)."""
    if request.param == "three_kernels":
        create = b.cser_create

        def create_three(*args, **kw):
            args = list(args)
            if len(args) >= 11:
                args[10] |= b.FLAG_THREE_KERNELS
            else:
                kw["flags"] = kw.get("flags", 0) | b.FLAG_THREE_KERNELS
            return create(*args, **kw)
        monkeypatch.setattr(b, "cser_create", create_three)
    return request.param


def _within(got, want, rtol, atol):
    return np.abs(got.astype(np.float64) - want) <= rtol * np.abs(want) + atol


# ------------------------------------------------------------------ masks
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_mask_kernel_bit_exact_all_configs(cfg):
    w = synth.CONFIGS[cfg]
    B = w.n_blocks
    out = torch.empty(B, dtype=torch.uint8, device=DEV)
    for seed in (0, 0xDEADBEEF12345678):
        for t in (1, 2, w.H, 99, 2**32 + 5):
            for which, R in ((STREAM_GRAD, w.R1), (STREAM_RESET, w.R2)):
                b.cser_grbs_mask(seed, t, which, 0, B, R, out)
                assert np.array_equal(out.cpu().numpy(), grbs_mask(seed, t, which, B, R)), (seed, t, which)
    # slab with global block ids
    b.cser_grbs_mask(3, 7, 0, 1000, min(B, 3000) - 1000, w.R1, out)
    assert np.array_equal(out[: min(B, 3000) - 1000].cpu().numpy(),
                          grbs_mask(3, 7, 0, min(B, 3000) - 1000, w.R1, block_begin=1000))


def test_mask_kernel_odd_ratios_and_R1():
    out = torch.empty(5001, dtype=torch.uint8, device=DEV)
    for R in (1, 3, 7, 1000, 2**31 + 1, 2**32 - 1):
        b.cser_grbs_mask(9, 4, 1, 0, 5001, R, out)
        assert np.array_equal(out.cpu().numpy(), grbs_mask(9, 4, 1, 5001, R))


def test_oracle_philox_matches_curand_library():
    """cuRAND's Philox4_32_10: key = seed, counter = (offset/4 as 64 bits, subsequence as 64 bits)."""
    L = ctypes.CDLL(os.path.join(ROOT, "tests", "libcurand_philox_check.so"))
    L.curand_philox_words.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_void_p]
    rng = np.random.default_rng(0)
    n = 4096
    seed = rng.integers(0, 2**63, n, dtype=np.int64)
    subseq = rng.integers(0, 2**63, n, dtype=np.int64)
    blockctr = rng.integers(0, 2**61, n, dtype=np.int64)
    seed[0] = subseq[0] = blockctr[0] = 0
    ts, tq, to = (torch.from_numpy(a).to(DEV) for a in (seed, subseq, blockctr * 4))
    out = torch.zeros(4 * n, dtype=torch.int32, device=DEV)
    rc = L.curand_philox_words(ts.data_ptr(), tq.data_ptr(), to.data_ptr(), out.data_ptr(), n, None)
    torch.cuda.synchronize()
    assert rc == 0
    got = out.cpu().numpy().view(np.uint32).reshape(n, 4)
    u = lambda a: a.astype(np.uint64)
    want = philox4x32_10(u(seed) & 0xFFFFFFFF, u(seed) >> 32, u(blockctr) & 0xFFFFFFFF, u(blockctr) >> 32,
                         u(subseq) & 0xFFFFFFFF, u(subseq) >> 32)
    assert np.array_equal(got, np.stack(want, 1))


# ------------------------------------------------------------------ small shapes, element by element
def _run_both(d, n, bs, R1, R2, H, eta, beta, steps, seed=3, masks=None, x0=None, grads=None, dtype=np.float32,
              flags=0, oracle=CSEROracle):
    rng = np.random.default_rng(1000 + d + n)
    x0 = rng.standard_normal(d).astype(np.float32) if x0 is None else x0
    opt = b.CSER(d, n, bs, R1, R2, H, eta, beta, seed, flags=flags)
    ref = oracle(d, n, bs, R1, R2, H, eta, beta, seed, dtype=dtype)
    opt.set_x0(torch.from_numpy(x0).to(DEV))
    ref.set_x0(x0)
    for t in range(1, steps + 1):
        g = (rng.standard_normal(d)[None, :] + 0.5 * rng.standard_normal((n, d))).astype(np.float32) \
            if grads is None else grads[t - 1]
        if masks is not None:
            mg, mr = masks[t - 1]
            opt.inject_masks(torch.tensor(mg, dtype=torch.uint8, device=DEV),
                             None if mr is None else torch.tensor(mr, dtype=torch.uint8, device=DEV))
            ref.inject_masks(mg, mr)
        opt.step(torch.from_numpy(g).to(DEV))
        ref.step(g)
        assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref.mask_g)
        if t >= H:      # the reset mask of the last reset step, also when read after later ordinary steps
            assert np.array_equal(opt.state(b.STATE_MASK_R).cpu().numpy(), ref.mask_r), t
    return opt, ref


SHAPES = [
    # d, n, bs, R1, R2, H, beta
    (4096 + 40, 8, 256, 4, 4, 4, 0.0),        # vector path, ragged last block
    (4096 + 40, 8, 256, 4, 2, 3, 0.9),
    (20_000, 16, 1024, 2, 2, 2, 0.9),         # several CTAs, n = 16
    (1001, 3, 7, 2, 2, 2, 0.9),               # scalar path: d and bs not multiples of 4
    (999, 2, 1000, 2, 2, 1, 0.0),             # B = 1, H = 1
    (130, 1, 4, 3, 5, 2, 0.9),                # single worker, odd ratios
    (2048, 5, 4, 1, 1, 3, 0.9),               # R = 1: everything selected, smallest vector block
    (8, 8, 4, 2, 2, 1, 0.5),                  # tiny
    (262_144 + 4, 8, 512, 32, 32, 8, 0.9),    # many tiles, tail of one vector column
]


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", SHAPES)
def test_small_shapes_equal_float32_oracle_exactly(d, n, bs, R1, R2, H, beta, launch_path):
    opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, beta, steps=13)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
        got = opt.state(which).cpu().numpy()
        want = getattr(ref, name)
        assert got.shape == want.shape
        bad = got != want
        assert not bad.any(), (name, int(bad.sum()), np.argwhere(bad)[:5])
    assert opt.t == 13
    opt.close()


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", SHAPES[:4])
def test_small_shapes_within_stated_tolerance_of_float64_oracle(d, n, bs, R1, R2, H, beta, launch_path):
    for steps, rtol, atol_rms in ((1, 1e-6, None), (100, 1e-4, 1e-4)):
        opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, beta, steps=steps, dtype=np.float64)
        for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
            got = opt.state(which).cpu().numpy()
            want = getattr(ref, name)
            atol = 1e-7 if atol_rms is None else atol_rms * float(np.sqrt((want**2).mean()))
            assert _within(got, want, rtol, atol).all(), (steps, name)
        opt.close()


@pytest.mark.parametrize("beta", [0.0, 0.5])
def test_hand_worked_example_on_gpu(beta):
    gold = read_hand_example()
    g = [np.array([[1, 2, -1, 0], [3, -2, 1, 4]], np.float32), np.array([[2, 2, 2, 2], [0, 4, -2, 6]], np.float32)]
    masks = [([1, 0], None), ([0, 1], [0, 1])]
    opt = b.CSER(4, 2, 2, 7, 7, 2, 0.5, beta, 0)
    opt.set_x0(torch.tensor([1, 2, 3, 4], dtype=torch.float32, device=DEV))
    for t in (1, 2):
        mg, mr = masks[t - 1]
        opt.inject_masks(torch.tensor(mg, dtype=torch.uint8, device=DEV),
                         None if mr is None else torch.tensor(mr, dtype=torch.uint8, device=DEV))
        opt.step(torch.from_numpy(g[t - 1]).to(DEV))
        for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
            got = opt.state(which).cpu().numpy()
            for i in range(2):
                assert np.array_equal(got[i], np.array(gold[(beta, t, name, i)], np.float32)), (t, name, i)
    opt.close()


def test_all_four_mask_combinations_on_one_reset_step(launch_path):
    """Blocks in neither / update only / reset only / both masks, vector and scalar paths."""
    for d, bs in ((64, 16), (62, 15)):
        B = n_blocks(d, bs)
        mg = [0, 1, 0, 1, 1][:B]
        mr = [0, 0, 1, 1, 0][:B]
        masks = [(mg, mr)] * 3
        opt, ref = _run_both(d, 4, bs, 2, 2, 1, 0.1, 0.9, steps=3, masks=masks)
        for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m")):
            assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), (d, name)
        opt.close()


# ------------------------------------------------------------------ full-size workloads
def _sample_blocks(w, ref_masks_g, ref_masks_r, rng, n_random):
    B = w.n_blocks
    blocks = {0, B - 1, B // 2}
    # blocks whose elements straddle a 2^31-element boundary of the flattened [n, d] index
    flat = 2**31
    while flat < w.n_workers * w.d:
        col = flat % w.d
        blocks.update({col // w.block_size, max(col // w.block_size - 1, 0)})
        flat += 2**31
    blocks.update(int(v) for v in rng.integers(0, B, n_random))
    for masks in (ref_masks_g, ref_masks_r):
        for m in masks:
            sel = np.flatnonzero(m)
            if sel.size:
                blocks.update(int(v) for v in rng.choice(sel, min(8, sel.size), replace=False))
    return np.array(sorted(blocks), dtype=np.int64)


def _cols_of(blocks, w):
    parts = [np.arange(bk * w.block_size, min((bk + 1) * w.block_size, w.d), dtype=np.int64) for bk in blocks]
    return np.concatenate(parts)


def _full_size_parity(cfg, steps=None, n_random=192, impl2=False, flags=0, ratios=None):
    w = synth.CONFIGS[cfg]
    if ratios is not None:                      # same shape, other (R1, R2, H)
        from dataclasses import replace
        w = replace(w, R1=ratios[0], R2=ratios[1], H=ratios[2])
    oracle = CSERImpl2Oracle if impl2 else CSEROracle
    steps = w.steps if steps is None else steps
    rng = np.random.default_rng(cfg)
    B = w.n_blocks
    masks_g = [grbs_mask(w.seed, t, STREAM_GRAD, B, w.R1) for t in range(1, steps + 1)]
    masks_r = [grbs_mask(w.seed, t, STREAM_RESET, B, w.R2) for t in range(1, steps + 1) if t % w.H == 0]
    blocks = _sample_blocks(w, masks_g[::max(1, steps // 8)], masks_r[::max(1, len(masks_r) // 8)], rng, n_random)
    cols = _cols_of(blocks, w)
    cols_dev = torch.from_numpy(cols).to(DEV)
    refs = {dt: oracle(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                       dtype=dt, cols=cols) for dt in (np.float32, np.float64)}
    opt = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                 flags=(b.FLAG_NO_ERROR_ARRAY if impl2 else 0) | flags)
    x0 = synth.x0(w, DEV)
    opt.set_x0(x0)
    x0_s = x0[cols_dev].cpu().numpy()
    for r in refs.values():
        r.set_x0(x0_s)
    g = torch.empty((w.n_workers, w.d), dtype=torch.float32, device=DEV)
    buf = torch.empty((w.n_workers, w.d), dtype=torch.float32, device=DEV)
    names = ((b.STATE_X, "x"),) + (() if impl2 else ((b.STATE_E, "e"),)) + (((b.STATE_M, "m"),) if w.beta else ())

    def compare(rtol, atol_abs, atol_rms):
        for which, name in names:
            b.cser_read_state(opt.h, which, buf)
            got = buf[:, cols_dev].cpu().numpy()
            want32, want64 = refs[np.float32].__dict__[name], refs[np.float64].__dict__[name]
            atol = atol_abs + atol_rms * float(np.sqrt((want64**2).mean()))
            assert _within(got, want64, rtol, atol).all(), (cfg, name, "float64 tolerance")
            bad = got != want32
            assert not bad.any(), (cfg, name, "float32 exact", int(bad.sum()))

    for t in range(1, steps + 1):
        synth.gradients(w, t, DEV, out=g)
        opt.step(g)
        g_s = g[:, cols_dev].cpu().numpy()
        for r in refs.values():
            r.step(g_s)
        if t == 1:
            compare(1e-6, 1e-7, 0.0)
        if t in (1, w.H, steps):
            assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), masks_g[t - 1]), t
    compare(1e-4, 0.0, 1e-4)
    if impl2:
        # implementation II: right after a reset the reset-selected blocks agree across workers exactly
        if steps % w.H == 0:
            b.cser_read_state(opt.h, b.STATE_X, buf)
            mr = torch.from_numpy(masks_r[-1]).to(DEV).bool()
            sel_cols = mr.repeat_interleave(w.block_size)[: w.d]
            assert (buf[:, sel_cols] - buf[0:1, sel_cols]).abs().max().item() == 0.0
        opt.close()
        del g, buf
        torch.cuda.empty_cache()
        return
    # properties that hold at any size, on the whole state: Lemma 1 and zero error after reset
    b.cser_read_state(opt.h, b.STATE_X, buf)
    b.cser_read_state(opt.h, b.STATE_E, g)
    diff = buf - g
    spread = (diff - diff[0:1]).abs().max().item()
    assert spread <= 1e-4 * max(1.0, buf.abs().max().item()), spread
    if steps % w.H == 0:
        mr = torch.from_numpy(masks_r[-1]).to(DEV).bool()
        sel_cols = mr.repeat_interleave(w.block_size)[: w.d]
        assert g[:, sel_cols].abs().max().item() == 0.0
    assert opt.t == steps
    opt.close()
    del g, buf
    torch.cuda.empty_cache()


def test_config1_full_vector_every_element(launch_path):
    """d = 2^20, n = 8, 20 steps: the whole state against the oracle, not a sample."""
    w = synth.CONFIGS[1]
    opt = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed)
    ref32 = CSEROracle(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed, dtype=np.float32)
    ref64 = CSEROracle(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed, dtype=np.float64)
    x0 = synth.x0(w, DEV)
    opt.set_x0(x0)
    ref32.set_x0(x0.cpu().numpy()), ref64.set_x0(x0.cpu().numpy())
    for t in range(1, w.steps + 1):
        g = synth.gradients(w, t, DEV)
        opt.step(g)
        gh = g.cpu().numpy()
        ref32.step(gh), ref64.step(gh)
        assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref32.mask_g)
        if t == 1:
            for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")):
                assert _within(opt.state(which).cpu().numpy(), getattr(ref64, name), 1e-6, 1e-7).all()
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")):
        got = opt.state(which).cpu().numpy()
        want = getattr(ref64, name)
        assert _within(got, want, 1e-4, 1e-4 * float(np.sqrt((want**2).mean()))).all()
        assert np.array_equal(got, getattr(ref32, name))
    with pytest.raises(b.CSERError):
        opt.state(b.STATE_M)                       # no momentum array when beta == 0
    opt.close()


@pytest.mark.parametrize("cfg", [2, 3, 4])
def test_full_size_configs_on_sampled_blocks(cfg):
    _full_size_parity(cfg)


@pytest.mark.parametrize("cfg,ratios", [(2, (4, 4, 2)), (5, (4, 8, 2))])
def test_full_size_shapes_with_many_selected_blocks_on_sampled_blocks(cfg, ratios):
    """The WRN-sized and the BERT-large-sized vector with a quarter of the blocks selected: every iteration
    goes through the single-launch kernel (the per-iteration rule), at full size, past 2^31 elements for the
    larger one; sampled whole blocks against the oracle, Lemma 1 and e = 0 after resets on the whole state."""
    _full_size_parity(cfg, steps=6, n_random=96, ratios=ratios)


def test_config5_bert_large_sized_on_sampled_blocks():
    """About 43 GB of state and gradients; 64-bit indexing (n*d > 2^31)."""
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2**30:
        pytest.skip("needs about 65 GB of free device memory")
    _full_size_parity(5, n_random=96)


# ------------------------------------------------------------------ special cases and implementation II
@pytest.mark.parametrize("d,n,bs,R2,H,beta", [(4096 + 40, 8, 256, 4, 1, 0.0), (4096 + 40, 8, 256, 2, 4, 0.9),
                                              (1001, 3, 7, 2, 2, 0.9), (20_000, 16, 1024, 1, 3, 0.0)])
def test_no_update_sync_special_cases_csea_and_cser_pl(d, n, bs, R2, H, beta, launch_path):
    """R1 = 0 (C2 = 0): CSEA when H = 1, CSER-PL otherwise (Appendix A.1)."""
    opt, ref = _run_both(d, n, bs, 0, R2, H, 0.1, beta, steps=13)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    assert not opt.state(b.STATE_MASK_G).any()
    if H == 1 and beta == 0.0:                      # the paper's own three-line CSEA form
        rng = np.random.default_rng(1000 + d + n)
        x0 = rng.standard_normal(d).astype(np.float32)
        csea = CSEAOracle(d, n, bs, R2, 0.1, 3)
        csea.set_x0(x0)
        for _ in range(13):
            csea.step((rng.standard_normal(d)[None, :] + 0.5 * rng.standard_normal((n, d))).astype(np.float32))
        got = opt.state(b.STATE_X).cpu().numpy()
        assert _within(got, csea.x, 1e-5, 1e-5).all()
    opt.close()


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", SHAPES)
def test_implementation_II_equals_its_float32_oracle_exactly(d, n, bs, R1, R2, H, beta, launch_path):
    opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, beta, steps=13, flags=b.FLAG_NO_ERROR_ARRAY,
                         oracle=CSERImpl2Oracle)
    for which, name in ((b.STATE_X, "x"),) + (((b.STATE_M, "m"),) if beta else ()):
        got, want = opt.state(which).cpu().numpy(), getattr(ref, name)
        bad = got != want
        assert not bad.any(), (name, int(bad.sum()), np.argwhere(bad)[:5])
    with pytest.raises(b.CSERError):
        opt.state(b.STATE_E)
    opt.close()


def test_implementation_II_models_match_implementation_I(launch_path):
    d, n, bs = 50_000 + 12, 8, 256
    a, ra = _run_both(d, n, bs, 4, 2, 4, 0.1, 0.9, steps=40)
    c, rc = _run_both(d, n, bs, 4, 2, 4, 0.1, 0.9, steps=40, flags=b.FLAG_NO_ERROR_ARRAY, oracle=CSERImpl2Oracle)
    xa, xc = a.state(b.STATE_X), c.state(b.STATE_X)
    assert (xa - xc).abs().max().item() <= 1e-4 * xa.abs().max().item()
    assert torch.equal(a.state(b.STATE_M), c.state(b.STATE_M))
    a.close(), c.close()


def test_all_four_mask_combinations_implementation_II():
    for d, bs in ((64, 16), (62, 15)):
        B = n_blocks(d, bs)
        masks = [([0, 1, 0, 1, 1][:B], [0, 0, 1, 1, 0][:B])] * 3
        opt, ref = _run_both(d, 4, bs, 2, 2, 1, 0.1, 0.9, steps=3, masks=masks, flags=b.FLAG_NO_ERROR_ARRAY,
                             oracle=CSERImpl2Oracle)
        for which, name in ((b.STATE_X, "x"), (b.STATE_M, "m")):
            assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), (d, name)
        opt.close()


def test_implementation_II_full_size_headline_workload_on_sampled_blocks():
    _full_size_parity(2, impl2=True)


# ------------------------------------------------------------------ exact-count GRBS
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_exact_count_masks_bit_exact_at_every_workload_size(cfg):
    """d = B (block_size 1... no: one element per block would be slow) - use 4-element blocks, one worker."""
    w = synth.CONFIGS[cfg]
    B = w.n_blocks
    opt = b.CSER(B * 4, 1, 4, w.R1, w.R2, 2, 0.1, 0.0, 77, flags=b.FLAG_EXACT_COUNT)
    g = torch.zeros((1, B * 4), device=DEV)
    for t in (1, 2, 3, 4):
        opt.step(g)
        mg = opt.state(b.STATE_MASK_G).cpu().numpy()
        assert int(mg.sum()) == exact_count(B, w.R1)
        assert np.array_equal(mg, grbs_mask_exact(77, t, STREAM_GRAD, B, w.R1)), (cfg, t)
        if t % 2 == 0:
            mr = opt.state(b.STATE_MASK_R).cpu().numpy()
            assert np.array_equal(mr, grbs_mask_exact(77, t, STREAM_RESET, B, w.R2)), (cfg, t)
    opt.close()


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", [(4096 + 40, 8, 256, 4, 4, 4, 0.0), (20_000, 16, 1024, 2, 2, 2, 0.9),
                                                 (1001, 3, 7, 2, 3, 2, 0.9), (999, 2, 1000, 2, 2, 1, 0.0),
                                                 (64, 2, 4, 64, 1, 1, 0.9), (262_144 + 4, 8, 512, 32, 32, 8, 0.9)])
def test_exact_count_mode_equals_its_float32_oracle_exactly(d, n, bs, R1, R2, H, beta):
    rng = np.random.default_rng(5)
    x0 = rng.standard_normal(d).astype(np.float32)
    opt = b.CSER(d, n, bs, R1, R2, H, 0.1, beta, 3, flags=b.FLAG_EXACT_COUNT)
    ref = CSEROracle(d, n, bs, R1, R2, H, 0.1, beta, 3, dtype=np.float32, exact_count=True)
    opt.set_x0(torch.from_numpy(x0).to(DEV)), ref.set_x0(x0)
    for t in range(1, 10):
        g = rng.standard_normal((n, d)).astype(np.float32)
        opt.step(torch.from_numpy(g).to(DEV)), ref.step(g)
        assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref.mask_g)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.close()
    assert not b.lib().cser_create_ex(100, 2, 4, 2, 2, 2, 0.1, 0.0, 0, 5, b.FLAG_EXACT_COUNT)   # slabs: not supported


# ------------------------------------------------------------------ more edges
@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta", [
    (4, 33, 4, 2, 2, 2, 0.9),          # one vector column, many workers (batches of 4 with a tail of 1)
    (3, 2, 8, 2, 2, 1, 0.0),           # shorter than one vector column: scalar path, block longer than d
    (1, 1, 1, 1, 1, 1, 0.9),           # the smallest problem there is
    (12, 7, 4, 1, 1, 5, 0.0),          # R = 1 without momentum, n not a multiple of the batch
    (40_000, 64, 128, 16, 8, 2, 0.9),  # many workers
    (1 << 16, 2, 1 << 16, 2, 2, 2, 0.9),   # a single huge block
])
def test_edge_shapes_equal_float32_oracle_exactly(d, n, bs, R1, R2, H, beta, launch_path):
    opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, beta, steps=7)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e")) + (((b.STATE_M, "m"),) if beta else ()):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.close()


def test_steps_on_a_side_stream_and_kernel_timing_hooks(launch_path):
    w = synth.CONFIGS[2].scaled(d=300_000, steps=6)
    side = torch.cuda.Stream()
    a = b.CSER(w.d, w.n_workers, w.block_size, 4, 2, 2, w.eta, w.beta, 8)
    c = b.CSER(w.d, w.n_workers, w.block_size, 4, 2, 2, w.eta, w.beta, 8)
    x0 = synth.x0(w, DEV)
    a.set_x0(x0), c.set_x0(x0)
    grads = [synth.gradients(w, t, DEV) for t in range(1, w.steps + 1)]
    torch.cuda.synchronize()
    n0 = b.cser_launch_count(c.h)
    b.cser_set_timing(c.h, True)
    for g in grads:
        a.step(g)
        with torch.cuda.stream(side):
            c.step(g)                                   # binding passes torch's current stream
            sel_ms, step_ms = b.cser_last_kernel_ms(c.h)
            assert 0.0 <= sel_ms < 50.0 and 0.0 < step_ms < 50.0
    side.synchronize()
    torch.cuda.synchronize()
    if launch_path == "three_kernels":
        # per step: selected-block kernel, streaming kernel and the NEXT step's select kernel; the first
        # step also runs its own select kernel
        assert b.cser_launch_count(c.h) - n0 == 3 * len(grads) + 1
    else:
        assert b.cser_launch_count(c.h) - n0 == len(grads)      # small problem: one kernel per step
    for which in (b.STATE_X, b.STATE_E, b.STATE_M):
        assert torch.equal(a.state(which), c.state(which))
    a.close(), c.close()


def test_learning_rate_schedule_and_column_reads(launch_path):
    d, n, bs = 10_000, 4, 64
    rng = np.random.default_rng(8)
    x0 = rng.standard_normal(d).astype(np.float32)
    opt = b.CSER(d, n, bs, 4, 2, 3, 0.1, 0.9, 6)
    opt.set_x0(torch.from_numpy(x0).to(DEV))
    ref = None
    x_ref = e_ref = m_ref = None
    lrs = [0.1, 0.1, 0.02, 0.02, 0.004, 0.004]
    state = None
    for t, lr in enumerate(lrs, 1):
        g = rng.standard_normal((n, d)).astype(np.float32)
        b.cser_set_lr(opt.h, lr)
        opt.step(torch.from_numpy(g).to(DEV))
        # oracle with the same schedule: a fresh oracle per learning rate, carrying the state over
        o = CSEROracle(d, n, bs, 4, 2, 3, lr, 0.9, 6, dtype=np.float32)
        o.set_x0(x0)
        if state is not None:
            o.x, o.e, o.m = state
        o.t = t - 1
        o.step(g)
        state = (o.x, o.e, o.m)
    assert np.array_equal(opt.state(b.STATE_X).cpu().numpy(), state[0])
    assert np.array_equal(opt.state(b.STATE_E).cpu().numpy(), state[1])
    # column window, to device and to host
    for dev in (DEV, "cpu"):
        win = torch.empty((n, 300), dtype=torch.float32, device=dev)
        b.cser_read_columns(opt.h, b.STATE_M, 9_700, 300, win)
        torch.cuda.synchronize()
        assert np.array_equal(win.cpu().numpy(), state[2][:, 9_700:])
    assert b.lib().cser_read_columns(opt.h, b.STATE_X, 9_900, 200, win.data_ptr(), win.numel(), None) == -1
    assert b.lib().cser_set_lr(opt.h, float("inf")) == -1
    opt.close()


def test_two_handles_stepping_concurrently_on_two_streams(launch_path):
    w = synth.CONFIGS[2].scaled(d=1_000_000, steps=12)
    seeds = (31, 32)
    ref = [b.CSER(w.d, w.n_workers, w.block_size, 8, 4, 3, w.eta, w.beta, s) for s in seeds]
    par = [b.CSER(w.d, w.n_workers, w.block_size, 8, 4, 3, w.eta, w.beta, s) for s in seeds]
    x0 = synth.x0(w, DEV)
    for h in ref + par:
        h.set_x0(x0)
    grads = [synth.gradients(w, t, DEV) for t in range(1, w.steps + 1)]
    torch.cuda.synchronize()
    for g in grads:                                   # one after the other
        for h in ref:
            h.step(g)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for g in grads:                                   # interleaved on two streams, no synchronization between
        for h, st in zip(par, streams):
            with torch.cuda.stream(st):
                h.step(g)
    torch.cuda.synchronize()
    for a, c in zip(ref, par):
        for which in (b.STATE_X, b.STATE_E, b.STATE_M):
            assert torch.equal(a.state(which), c.state(which))
    [h.close() for h in ref + par]


def test_l2_resident_state_gives_the_same_results(launch_path):
    w = synth.CONFIGS[1].scaled(d=300_000, steps=9)          # 9.6 MB of state: fits the L2 set-aside
    a = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 3)
    c = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 3, flags=b.FLAG_L2_RESIDENT)
    big = b.CSER(30_000_000, 8, 256, 4, 4, 4, 0.1, 0.0, 3, flags=b.FLAG_L2_RESIDENT)   # 1.9 GB: flag ignored
    x0 = synth.x0(w, DEV)
    a.set_x0(x0), c.set_x0(x0)
    for t in range(1, w.steps + 1):
        g = synth.gradients(w, t, DEV)
        a.step(g), c.step(g)
    big.step(torch.zeros((8, 30_000_000), device=DEV))
    for which in (b.STATE_X, b.STATE_E):
        assert torch.equal(a.state(which), c.state(which))
    # two L2-resident handles share the context's set-aside: destroying one leaves the other's in place
    c2 = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 3, flags=b.FLAG_L2_RESIDENT)
    c2.set_x0(x0)
    c.close()
    a2 = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 3)
    a2.set_x0(x0)
    for t in range(1, 6):
        g = synth.gradients(w, t, DEV)
        a2.step(g), c2.step(g)
    for which in (b.STATE_X, b.STATE_E):
        assert torch.equal(a2.state(which), c2.state(which))
    a.close(), a2.close(), c2.close(), big.close()


def test_misaligned_gradient_pointer_takes_the_scalar_path():
    d, n = 1024, 4
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal(d).astype(np.float32)
    opt = b.CSER(d, n, 64, 2, 2, 2, 0.1, 0.9, 4)
    ref = CSEROracle(d, n, 64, 2, 2, 2, 0.1, 0.9, 4, dtype=np.float32)
    opt.set_x0(torch.from_numpy(x0).to(DEV)), ref.set_x0(x0)
    buf = torch.zeros(n * d + 1, device=DEV)
    for _ in range(4):
        g = rng.standard_normal((n, d)).astype(np.float32)
        view = buf[1:].view(n, d)                      # 4-byte aligned only
        view.copy_(torch.from_numpy(g))
        assert view.data_ptr() % 16 == 4
        b.cser_step(opt.h, view)
        ref.step(g)
    assert np.array_equal(opt.state(b.STATE_X).cpu().numpy(), ref.x)
    assert np.array_equal(opt.state(b.STATE_E).cpu().numpy(), ref.e)
    opt.close()


# ------------------------------------------------------------------ replayable steps and CUDA graphs
@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta,flags", [
    (4096 + 40, 8, 256, 4, 2, 3, 0.9, 0), (1001, 3, 7, 2, 3, 2, 0.0, 0), (50_000, 16, 512, 8, 4, 1, 0.9, 0),
    (20_000, 4, 64, 1, 2, 4, 0.9, 0), (30_000, 8, 128, 0, 2, 2, 0.0, 0), (30_000, 8, 128, 4, 4, 2, 0.9, 1)])
def test_replayable_steps_equal_ordinary_steps_and_the_oracle(d, n, bs, R1, R2, H, beta, flags, launch_path):
    """cser_step, then replayable steps (not captured), then cser_step again: one trajectory."""
    rng = np.random.default_rng(77)
    x0 = rng.standard_normal(d).astype(np.float32)
    impl2 = bool(flags & b.FLAG_NO_ERROR_ARRAY)
    opt = b.CSER(d, n, bs, R1, R2, H, 0.1, beta, 12, flags=flags)
    ref = (CSERImpl2Oracle if impl2 else CSEROracle)(d, n, bs, R1, R2, H, 0.1, beta, 12, dtype=np.float32)
    opt.set_x0(torch.from_numpy(x0).to(DEV)), ref.set_x0(x0)
    for phase, steps in (("plain", 3), ("replay", 7), ("plain", 3)):
        if phase == "replay":
            b.cser_replay_begin(opt.h)
        for _ in range(steps):
            g = rng.standard_normal((n, d)).astype(np.float32)
            gd = torch.from_numpy(g).to(DEV)
            if phase == "replay":
                b.cser_step_replayable(opt.h, gd)
            else:
                opt.step(gd)
            ref.step(g)
            assert opt.t == ref.t
            assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref.mask_g), (phase, ref.t)
        if phase == "replay":
            assert b.lib().cser_step(opt.h, gd.data_ptr(), None) == -1         # refused in between
            b.cser_replay_end(opt.h)
    names = ((b.STATE_X, "x"),) + (() if impl2 else ((b.STATE_E, "e"),)) + (((b.STATE_M, "m"),) if beta else ())
    for which, name in names:
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.close()


def test_step_captured_once_in_a_cuda_graph_and_replayed(launch_path):
    w = synth.CONFIGS[2].scaled(d=400_000 + 8, steps=20)
    R1, R2, H = 4, 2, 3
    opt = b.CSER(w.d, w.n_workers, w.block_size, R1, R2, H, w.eta, w.beta, 21)
    ref = CSEROracle(w.d, w.n_workers, w.block_size, R1, R2, H, w.eta, w.beta, 21, dtype=np.float32)
    x0 = synth.x0(w, DEV)
    opt.set_x0(x0), ref.set_x0(x0.cpu().numpy())
    grads = [synth.gradients(w, t, DEV) for t in range(1, w.steps + 1)]
    static_g = torch.empty_like(grads[0])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b.cser_replay_begin(opt.h)
        static_g.copy_(grads[0])
        b.cser_step_replayable(opt.h, static_g)                 # iteration 1, eagerly (also warms up)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
        b.cser_step_replayable(opt.h, static_g)                 # captured, not run
    ref.step(grads[0].cpu().numpy())
    for t in range(2, w.steps + 1):
        static_g.copy_(grads[t - 1])
        graph.replay()
        ref.step(grads[t - 1].cpu().numpy())
    torch.cuda.synchronize()
    assert opt.t == w.steps                                      # read from the device
    b.cser_replay_end(opt.h)
    assert opt.t == w.steps
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m")):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.step(grads[0])                                           # ordinary steps continue from there
    ref.step(grads[0].cpu().numpy())
    assert np.array_equal(opt.state(b.STATE_X).cpu().numpy(), ref.x)
    opt.close()


@pytest.mark.parametrize("n_plain,n_replay", [(3, 2), (2, 2), (4, 4), (1, 1)])
def test_reset_mask_of_the_last_reset_step_stays_readable_around_replay_mode(n_plain, n_replay, launch_path):
    """CSER_STATE_MASK_R is the reset mask of the last reset step that was executed - also when replay mode
    ends one step before a reset (its select kernel has then already prepared the next reset mask), when no
    reset ran during replay, and on the ordinary steps that follow."""
    d, n, bs, R1, R2, H = 4096 + 40, 4, 64, 4, 2, 3
    rng = np.random.default_rng(3)
    opt = b.CSER(d, n, bs, R1, R2, H, 0.1, 0.9, 17)
    ref = CSEROracle(d, n, bs, R1, R2, H, 0.1, 0.9, 17, dtype=np.float32)
    x0 = rng.standard_normal(d).astype(np.float32)
    opt.set_x0(torch.from_numpy(x0).to(DEV)), ref.set_x0(x0)
    g = torch.empty((n, d), device=DEV)

    def check(t):
        if t >= H:
            assert np.array_equal(opt.state(b.STATE_MASK_R).cpu().numpy(), ref.mask_r), t
        assert np.array_equal(opt.state(b.STATE_X).cpu().numpy(), ref.x), t

    t = 0
    for _ in range(n_plain):
        t += 1
        g.copy_(torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)))
        opt.step(g), ref.step(g.cpu().numpy())
        check(t)
    b.cser_replay_begin(opt.h)
    for _ in range(n_replay):
        t += 1
        g.copy_(torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)))
        b.cser_step_replayable(opt.h, g), ref.step(g.cpu().numpy())
        check(t)
    b.cser_replay_end(opt.h)
    check(t)
    for _ in range(4):
        t += 1
        g.copy_(torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)))
        opt.step(g), ref.step(g.cpu().numpy())
        check(t)
    opt.close()


# ------------------------------------------------------------------ randomized differential test
def test_random_shapes_parameters_and_flags_against_the_float32_oracle():
    """400 random problems (shape, ratios, reset interval, momentum, flags, injected masks now and
    then, host-gradient entry now and then): the state must equal the float32 oracle exactly."""
    rng = np.random.default_rng(20240607)
    for case in range(400):
        n = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 16, 17, 33]))
        bs = int(rng.choice([1, 3, 4, 8, 12, 16, 60, 64, 100, 128, 256, 1024]))
        d = int(rng.integers(1, 40)) * bs + int(rng.integers(0, bs)) if rng.random() < 0.7 else int(rng.integers(1, 3000))
        R1 = int(rng.choice([0, 1, 2, 3, 4, 7, 32]))
        R2 = int(rng.choice([1, 2, 3, 4, 16]))
        H = int(rng.integers(1, 5))
        beta = float(rng.choice([0.0, 0.5, 0.9]))
        eta = float(rng.choice([0.1, 0.01, 1.0]))
        impl2 = rng.random() < 0.3
        exact = rng.random() < 0.3
        seed = int(rng.integers(0, 2**62))
        flags = (b.FLAG_NO_ERROR_ARRAY if impl2 else 0) | (b.FLAG_EXACT_COUNT if exact else 0)
        flags |= b.FLAG_THREE_KERNELS if rng.random() < 0.4 else 0
        flags |= b.FLAG_STAGED_SELECTED if rng.random() < 0.3 else 0     # (implies the three kernels)
        opt = b.CSER(d, n, bs, R1, R2, H, eta, beta, seed, flags=flags)
        ref = (CSERImpl2Oracle if impl2 else CSEROracle)(d, n, bs, R1, R2, H, eta, beta, seed, dtype=np.float32,
                                                         exact_count=exact)
        x0 = rng.standard_normal(d).astype(np.float32)
        opt.set_x0(torch.from_numpy(x0).to(DEV) if rng.random() < 0.5 else torch.from_numpy(x0))
        ref.set_x0(x0)
        B = n_blocks(d, bs)
        label = (case, d, n, bs, R1, R2, H, beta, flags)
        for t in range(1, int(rng.integers(3, 9))):
            g = rng.standard_normal((n, d)).astype(np.float32)
            if rng.random() < 0.15:                    # injected masks for this step
                mg = rng.integers(0, 2, B).astype(np.uint8)
                mr = rng.integers(0, 2, B).astype(np.uint8)
                opt.inject_masks(torch.from_numpy(mg).to(DEV), torch.from_numpy(mr).to(DEV))
                ref.inject_masks(mg, mr)
            if rng.random() < 0.2:
                opt.step_host(torch.from_numpy(g).pin_memory())
            else:
                opt.step(torch.from_numpy(g).to(DEV))
            ref.step(g)
            assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref.mask_g), label + (t, "mask")
        names = ((b.STATE_X, "x"),) + (() if impl2 else ((b.STATE_E, "e"),)) + (((b.STATE_M, "m"),) if beta else ())
        for which, name in names:
            got, want = opt.state(which).cpu().numpy(), getattr(ref, name)
            assert np.array_equal(got, want), label + (name, int((got != want).sum()))
        opt.close()


@pytest.mark.parametrize("R1,R2,H", [(16, 16, 2), (4, 4, 3), (16, 2, 2), (64, 64, 2)])
def test_large_problems_switch_between_one_launch_and_three_kernels_step_by_step(R1, R2, H):
    """Above 256 MB per step the launch path is chosen per iteration from the expected share of selected
    blocks (one launch from 1/4 on ordinary steps and from 1/10 on reset steps): (16, 16) and (16, 2)
    alternate between the paths, (4, 4) is all one launch, (64, 64) all three kernels.  Whatever the mix, masks
    and state must equal the float32 oracle's, and the reset mask must stay readable."""
    d, n, bs = 1_300_000 + 4, 8, 512
    assert n * d * 28 > 1 << 28
    opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, 0.9, steps=7)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m")):
        got, want = opt.state(which).cpu().numpy(), getattr(ref, name)
        assert np.array_equal(got, want), (name, int((got != want).sum()))
    opt.close()


# ------------------------------------------------------------------ the opt-in staged selected-block kernel
STAGED_SHAPES = [
    # d, n, bs, R1, R2, H, beta, flags
    (4096 + 40, 8, 256, 4, 4, 4, 0.0, 0),             # ragged last block
    (4096 + 40, 8, 256, 4, 2, 3, 0.9, 0),
    (20_000, 16, 1024, 2, 2, 2, 0.9, 0),              # n = 16: blocks cut into several chunks
    (262_144 + 4, 8, 512, 32, 32, 8, 0.9, 0),         # the headline shape's geometry, tail of one vector column
    (60_000, 8, 2048, 1, 1, 2, 0.9, 0),               # R = 1: dense walk, every block update- and reset-selected
    (33_000, 3, 64, 2, 3, 1, 0.5, 0),                 # smallest staged block (16 vector columns), odd worker count
    (50_000, 8, 512, 3, 2, 2, 0.9, 1),                # implementation II (no error array)
    (50_000, 5, 512, 0, 2, 1, 0.0, 1),                # CSEA, implementation II, no momentum
    (70_000, 24, 4096, 2, 2, 2, 0.9, 0),              # many workers: a stage holds 32 columns
]


@pytest.mark.parametrize("d,n,bs,R1,R2,H,beta,flags", STAGED_SHAPES)
def test_staged_selected_block_kernel_equals_float32_oracle_exactly(d, n, bs, R1, R2, H, beta, flags):
    """CSER_FLAG_STAGED_SELECTED: the shared-memory staged kernel must give the same bits as the oracle
    (and hence as the default kernel) on update-selected, reset-selected and doubly selected blocks."""
    impl2 = bool(flags & b.FLAG_NO_ERROR_ARRAY)
    opt, ref = _run_both(d, n, bs, R1, R2, H, 0.1, beta, steps=9, flags=flags | b.FLAG_STAGED_SELECTED,
                         oracle=CSERImpl2Oracle if impl2 else CSEROracle)
    names = ((b.STATE_X, "x"),) + (() if impl2 else ((b.STATE_E, "e"),)) + (((b.STATE_M, "m"),) if beta else ())
    for which, name in names:
        got, want = opt.state(which).cpu().numpy(), getattr(ref, name)
        assert np.array_equal(got, want), (name, int((got != want).sum()))
    opt.close()


@pytest.mark.parametrize("cfg", [2, 3])
def test_staged_kernel_full_size_on_sampled_blocks(cfg):
    """The opt-in staged kernel at full size in the launch configuration `bench.py --staged` times: the
    WRN-sized workload (blocks in one chunk) and the ResNet-50-sized one (n = 16: blocks cut into chunks)."""
    _full_size_parity(cfg, steps=16, flags=b.FLAG_STAGED_SELECTED)


def test_staged_kernel_with_injected_masks_replay_and_host_gradients():
    """The staged kernel behind the other entry points: injected masks (all four combinations), replayable
    steps (reset flag and list length read on the device) and host-gradient slabs (column ranges)."""
    d, n, bs = 64 * 40 + 20, 4, 64
    B = n_blocks(d, bs)
    rng = np.random.default_rng(5)
    masks = [(rng.integers(0, 2, B).astype(np.uint8), rng.integers(0, 2, B).astype(np.uint8)) for _ in range(4)]
    opt, ref = _run_both(d, n, bs, 2, 2, 1, 0.1, 0.9, steps=4, masks=masks, flags=b.FLAG_STAGED_SELECTED)
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m")):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.close()
    w = synth.CONFIGS[2].scaled(d=1_200_000 + 4, steps=6)
    a = b.CSER(w.d, w.n_workers, w.block_size, 4, 2, 3, w.eta, w.beta, 5, flags=b.FLAG_STAGED_SELECTED)
    c = b.CSER(w.d, w.n_workers, w.block_size, 4, 2, 3, w.eta, w.beta, 5)
    x0 = synth.x0(w, DEV)
    a.set_x0(x0), c.set_x0(x0)
    pinned = torch.empty((w.n_workers, w.d), dtype=torch.float32).pin_memory()
    for t in range(1, w.steps + 1):
        g = synth.gradients(w, t, DEV)
        pinned.copy_(g)
        if t == 3:
            b.cser_replay_begin(a.h)
            b.cser_step_replayable(a.h, g)
            b.cser_replay_end(a.h)
        elif t % 2:
            a.step(g)
        else:
            a.step_host(pinned)
        c.step(g)
        torch.cuda.synchronize()
    for which in (b.STATE_X, b.STATE_E, b.STATE_M):
        assert torch.equal(a.state(which), c.state(which)), which
    a.close(), c.close()


def test_a_staged_kernel_wait_that_runs_out_is_reported_and_nothing_hangs():
    """The staged kernel's waits on its shared-memory barriers are bounded.  One CTA is told to expect bytes
    that never arrive (test hook) with the limit lowered to 0.1 s: the kernel must end by itself, the handle
    must report the failure on every later call, and the CUDA context must stay usable (another handle steps
    on, a plain copy works)."""
    import time
    L = b.lib()
    d, n, bs = 64 * 300, 4, 64
    bad = b.CSER(d, n, bs, 2, 2, 2, 0.1, 0.9, 3, flags=b.FLAG_STAGED_SELECTED)
    good = b.CSER(d, n, bs, 2, 2, 2, 0.1, 0.9, 3, flags=b.FLAG_STAGED_SELECTED)
    x0 = torch.randn(d, device=DEV)
    bad.set_x0(x0), good.set_x0(x0)
    g = torch.randn((n, d), device=DEV)
    bad.step(g), good.step(g)
    torch.cuda.synchronize()
    assert L.cser_debug_stall_next_staged_step(bad.h, 200) == 0
    t0 = time.perf_counter()
    bad.step(g)                                        # enqueues the stalled kernel
    torch.cuda.synchronize()                           # ... which ends by itself
    assert time.perf_counter() - t0 < 10.0
    assert L.cser_step(bad.h, ctypes.c_void_p(g.data_ptr()), None) == -3
    assert "wait ran out" in b.cser_last_error()
    out = torch.empty((n, d), device=DEV)
    assert L.cser_read_state(bad.h, b.STATE_X, ctypes.c_void_p(out.data_ptr()), out.numel() * 4, None) == -3
    good.step(g)                                       # the context is fine
    torch.cuda.synchronize()
    assert bool(torch.isfinite(good.state(b.STATE_X)).all())
    assert torch.equal(g.clone(), g)
    h = bad.h
    bad.h = None
    torch.cuda.synchronize()
    b.cser_destroy(h)
    good.close()


# ------------------------------------------------------------------ C2 = 0 without an error array
@pytest.mark.parametrize("H,R2,beta", [(1, 4, 0.0), (1, 2, 0.9), (4, 2, 0.9), (3, 1, 0.0)])
def test_csea_and_cser_pl_in_implementation_II(H, R2, beta, launch_path):
    """R1 = 0 together with CSER_FLAG_NO_ERROR_ARRAY: the special cases of Appendix A.1 (CSEA for H = 1,
    CSER-PL otherwise) in the form without an error array of Appendix A.4: nothing is exchanged between
    resets and a reset replaces the reset-selected blocks of x by their mean over workers."""
    d, n, bs = 4096 + 40, 8, 256
    opt, ref = _run_both(d, n, bs, 0, R2, H, 0.1, beta, steps=9, flags=b.FLAG_NO_ERROR_ARRAY,
                         oracle=CSERImpl2Oracle)
    assert np.array_equal(opt.state(b.STATE_X).cpu().numpy(), ref.x)
    if beta:
        assert np.array_equal(opt.state(b.STATE_M).cpu().numpy(), ref.m)
    # the models agree with implementation I's (same masks, same gradients) to rounding
    one, ref1 = _run_both(d, n, bs, 0, R2, H, 0.1, beta, steps=9)
    x2, x1 = opt.state(b.STATE_X).cpu().numpy().astype(np.float64), one.state(b.STATE_X).cpu().numpy().astype(np.float64)
    assert np.abs(x2 - x1).max() <= 1e-4 * np.abs(x1).max()
    if R2 == 1:     # delta_1 = 1: every reset makes all workers' models equal (local SGD with period H)
        x = opt.state(b.STATE_X).cpu().numpy()
        assert (x == x[0]).all()
    opt.close(), one.close()


# ------------------------------------------------------------------ boundary behaviour
def test_host_gradient_entry_point_equals_device_entry_point(launch_path):
    w = synth.CONFIGS[2].scaled(d=3_000_000 + 4, steps=10)
    a = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 5)
    c = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, 5)
    x0 = synth.x0(w, DEV)
    a.set_x0(x0), c.set_x0(x0.cpu())             # x0 from device and from host memory
    pinned = torch.empty((w.n_workers, w.d), dtype=torch.float32).pin_memory()
    for t in range(1, w.steps + 1):
        g = synth.gradients(w, t, DEV)
        pinned.copy_(g)
        a.step(g)
        c.step_host(pinned)
        torch.cuda.synchronize()
    for which in (b.STATE_X, b.STATE_E, b.STATE_M, b.STATE_MASK_G, b.STATE_MASK_R):
        assert torch.equal(a.state(which), c.state(which))
    a.close(), c.close()


def test_column_slabs_reproduce_the_whole_vector(launch_path):
    """Two handles that each own a slab of whole blocks, with global block ids, and exchange nothing."""
    from paper_2007_13221_b200.shard import slab_of_rank
    w = synth.CONFIGS[3].scaled(d=100_000 + 8, steps=9)
    whole = b.CSER(w.d, w.n_workers, w.block_size, 4, 2, w.H, w.eta, w.beta, 1)
    x0 = synth.x0(w, DEV)
    whole.set_x0(x0)
    slabs = []
    for r in range(2):
        c0, c1, b0 = slab_of_rank(w.d, w.block_size, r, 2)
        s = b.CSER(c1 - c0, w.n_workers, w.block_size, 4, 2, w.H, w.eta, w.beta, 1, block_begin=b0)
        s.set_x0(x0[c0:c1].contiguous())
        slabs.append((c0, c1, s))
    for t in range(1, w.steps + 1):
        g = synth.gradients(w, t, DEV)
        whole.step(g)
        for c0, c1, s in slabs:
            s.step(g[:, c0:c1].contiguous())
    for which in (b.STATE_X, b.STATE_E, b.STATE_M):
        full = whole.state(which)
        for c0, c1, s in slabs:
            assert torch.equal(full[:, c0:c1], s.state(which))
    whole.close()
    [s.close() for _, _, s in slabs]


def test_checkpoint_and_resume_is_bit_identical(launch_path):
    w = synth.CONFIGS[2].scaled(d=50_000, steps=30)
    a = b.CSER(w.d, w.n_workers, w.block_size, 4, 4, w.H, w.eta, w.beta, 2)
    a.set_x0(synth.x0(w, DEV))
    for t in range(1, 11):
        a.step(synth.gradients(w, t, DEV))
    snap = {k: a.state(k).clone() for k in (b.STATE_X, b.STATE_E, b.STATE_M)}
    t_snap = a.t
    for t in range(11, 21):
        a.step(synth.gradients(w, t, DEV))
    final = {k: a.state(k).clone() for k in (b.STATE_X, b.STATE_E, b.STATE_M)}
    c = b.CSER(w.d, w.n_workers, w.block_size, 4, 4, w.H, w.eta, w.beta, 2)
    for k, v in snap.items():
        b.cser_write_state(c.h, k, v)
    b.cser_write_state(c.h, b.STATE_T, torch.tensor([t_snap], dtype=torch.int64))
    for t in range(11, 21):
        c.step(synth.gradients(w, t, DEV))
    for k in final:
        assert torch.equal(final[k], c.state(k))
    a.close(), c.close()


def test_step_counter_across_the_32_bit_boundary(launch_path):
    """t is a 64-bit counter and enters the Philox counter as two 32-bit words: steps t = 2^32 - 1 .. 2^32 + 3
    (the counter restored with cser_write_state) must draw the oracle's masks and give its state, on both
    launch paths and in replay mode."""
    d, n, bs, R1, R2, H = 4096 + 40, 4, 64, 4, 2, 2
    t0 = 2**32 - 2
    rng = np.random.default_rng(11)
    x0 = rng.standard_normal(d).astype(np.float32)
    opt = b.CSER(d, n, bs, R1, R2, H, 0.1, 0.9, 5)
    ref = CSEROracle(d, n, bs, R1, R2, H, 0.1, 0.9, 5, dtype=np.float32)
    opt.set_x0(torch.from_numpy(x0).to(DEV)), ref.set_x0(x0)
    b.cser_write_state(opt.h, b.STATE_T, torch.tensor([t0], dtype=torch.int64))
    ref.t = t0
    for k in range(1, 8):
        g = rng.standard_normal((n, d)).astype(np.float32)
        gd = torch.from_numpy(g).to(DEV)
        if k == 5:
            b.cser_replay_begin(opt.h)
            b.cser_step_replayable(opt.h, gd)
            b.cser_replay_end(opt.h)
        else:
            opt.step(gd)
        ref.step(g)
        assert opt.t == t0 + k
        assert np.array_equal(opt.state(b.STATE_MASK_G).cpu().numpy(), ref.mask_g), k
    for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m")):
        assert np.array_equal(opt.state(which).cpu().numpy(), getattr(ref, name)), name
    opt.close()


def test_errors_are_reported_not_raised_on_the_device():
    L = b.lib()
    assert not L.cser_create(0, 8, 256, 4, 4, 4, 0.1, 0.0, 0)
    assert "positive" in b.cser_last_error()
    assert not L.cser_create(100, 8, 256, 4, 0, 4, 0.1, 0.0, 0)          # R2 = 0: delta_1 must be positive
    assert not L.cser_create_ex(100, 8, 256, 4, 4, 4, 0.1, 0.0, 0, 0, 0x80)  # unknown flag
    assert not L.cser_create(100, 8, 256, 4, 4, 0, 0.1, 0.0, 0)
    assert not L.cser_create(100, 8, 256, 4, 4, 4, float("nan"), 0.0, 0)
    assert not L.cser_create(100, 8, 256, 4, 4, 4, 0.1, 1.0, 0)
    assert L.cser_step(None, None, None) == -1
    opt = b.CSER(100, 2, 10, 2, 2, 2, 0.1, 0.0, 0)
    assert L.cser_step(opt.h, None, None) == -1
    host = torch.zeros((2, 100))
    assert L.cser_step(opt.h, ctypes.c_void_p(host.data_ptr()), None) == -1      # host pointer
    assert "device memory" in b.cser_last_error()
    small = torch.zeros(10, device=DEV)
    assert L.cser_read_state(opt.h, b.STATE_X, ctypes.c_void_p(small.data_ptr()), 40, None) == -4
    assert L.cser_read_state(opt.h, b.STATE_M, ctypes.c_void_p(small.data_ptr()), 40, None) == -1
    assert L.cser_read_state(opt.h, 17, ctypes.c_void_p(small.data_ptr()), 40, None) == -1
    dev_g = torch.zeros((2, 100 + 1), device=DEV)
    assert L.cser_step(opt.h, ctypes.c_void_p(dev_g.data_ptr() + 2), None) == -1    # not 4-byte aligned
    assert "aligned" in b.cser_last_error()
    assert L.cser_write_state(opt.h, b.STATE_X, ctypes.c_void_p(small.data_ptr()), 40, None) == -4
    assert L.cser_write_state(opt.h, b.STATE_MASK_G, ctypes.c_void_p(small.data_ptr()), 10, None) == -1
    assert L.cser_debug_set_masks(opt.h, None, None, None) == -1
    assert L.cser_set_x0(opt.h, None, None) == -1
    assert L.cser_grbs_mask(0, 1, 2, 0, 10, 4, ctypes.c_void_p(small.data_ptr()), None) == -1   # bad compressor id
    assert L.cser_last_kernel_ms(opt.h, None, None) == -1                                # nothing timed yet
    assert opt.t == 0                                 # failed calls did not advance the step counter
    opt.step(torch.zeros((2, 100), device=DEV))
    assert opt.t == 1
    opt.close()


def test_refused_steps_leave_the_counter_and_the_state_alone(launch_path):
    """A step that is refused (bad pointer, wrong kind of memory, misaligned) happens before the iteration
    counter moves: interleaved with good steps it must leave t, the masks and the state exactly as on a
    handle that never saw it."""
    L = b.lib()
    d, n, bs = 5000, 4, 64
    a = b.CSER(d, n, bs, 4, 2, 2, 0.1, 0.9, 9)
    c = b.CSER(d, n, bs, 4, 2, 2, 0.1, 0.9, 9)
    x0 = torch.randn(d, device=DEV)
    a.set_x0(x0), c.set_x0(x0)
    host = torch.zeros((n, d))
    odd = torch.zeros(n * d + 1, device=DEV)
    for t in range(1, 7):
        g = torch.randn((n, d), device=DEV)
        assert L.cser_step(a.h, None, None) == -1
        assert L.cser_step(a.h, ctypes.c_void_p(host.data_ptr()), None) == -1
        assert L.cser_step(a.h, ctypes.c_void_p(odd.data_ptr() + 2), None) == -1
        assert a.t == t - 1
        a.step(g), c.step(g)
        assert a.t == c.t == t
    for which in (b.STATE_X, b.STATE_E, b.STATE_M, b.STATE_MASK_G, b.STATE_MASK_R):
        assert torch.equal(a.state(which), c.state(which)), which
    a.close(), c.close()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs a second GPU to own the foreign buffer")
def test_a_buffer_of_another_gpu_is_refused_before_anything_is_launched():
    """Device memory of another GPU passes a plain "is this device memory" check but would be dereferenced by
    kernels of this GPU; it must be refused on the host (nothing is launched on it)."""
    L = b.lib()
    opt = b.CSER(1000, 2, 10, 2, 2, 2, 0.1, 0.0, 0)
    foreign = torch.zeros((2, 1000), device="cuda:1")
    torch.cuda.set_device(0)
    assert L.cser_step(opt.h, ctypes.c_void_p(foreign.data_ptr()), None) == -1
    assert "lives on device" in b.cser_last_error()
    assert opt.t == 0
    opt.close()
