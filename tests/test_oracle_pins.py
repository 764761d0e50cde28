"""Pins of the CPU oracle to facts fixed by the paper and by mathematics.

None of these tests touches the CUDA library.  Each one would fail for some
plausible mistake in the oracle (dropped term, wrong sign, wrong index,
transposed operand), and none re-types the oracle's own formula.
"""
import os
import subprocess
import sys
from fractions import Fraction

import numpy as np
import pytest

from _golden import read_hand_example

from oracle import (CSEAOracle, CSEROracle, CSERImpl2Oracle, exact_count, grbs_mask, grbs_mask_exact, n_blocks, philox4_generic,
                    philox4x32_10, psync, STREAM_GRAD, STREAM_RESET)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


# --------------------------------------------------------------------------- Philox
def test_philox_round_structure_matches_numpy_philox4x64():
    """NumPy ships Philox4x64-10; the generic routine at W = 64 must reproduce it.
    (NumPy increments the counter once before producing its first block.)"""
    rng = np.random.default_rng(1)
    for _ in range(20):
        key = [int(v) for v in rng.integers(0, 2**63, 2)]
        ctr = [int(v) for v in rng.integers(0, 2**63, 4)]
        bg = np.random.Philox(key=np.array(key, np.uint64), counter=np.array(ctr, np.uint64))
        want = [int(v) for v in bg.random_raw(4)]
        got = philox4_generic(64, key, [ctr[0] + 1, ctr[1], ctr[2], ctr[3]])
        assert got == want


def test_philox_vectorised_32_equals_generic_32():
    rng = np.random.default_rng(2)
    args = rng.integers(0, 2**32, size=(6, 2000), dtype=np.uint64)
    out = philox4x32_10(*args)
    for s in range(0, 2000, 37):
        k0, k1, c0, c1, c2, c3 = (int(a[s]) for a in args)
        assert [int(w[s]) for w in out] == philox4_generic(32, [k0, k1], [c0, c1, c2, c3])
    # edge words
    for k in ([0, 0], [0xFFFFFFFF, 0xFFFFFFFF]):
        for c in ([0, 0, 0, 0], [0xFFFFFFFF] * 4):
            assert [int(w) for w in philox4x32_10(*k, *c)] == philox4_generic(32, k, c)


_TRITON_SNIPPET = r"""
import os, sys
os.environ["TRITON_INTERPRET"] = "1"
import torch, triton, triton.language as tl
@triton.jit
def k(out, seed, c0, c1, c2, c3):
    z = tl.arange(0, 1)
    a, b, c, d = tl.philox(seed, tl.full((1,), c0, tl.uint32), tl.full((1,), c1, tl.uint32),
                           tl.full((1,), c2, tl.uint32), tl.full((1,), c3, tl.uint32))
    tl.store(out + z, a); tl.store(out + 1 + z, b); tl.store(out + 2 + z, c); tl.store(out + 3 + z, d)
for line in sys.stdin:
    seed, c0, c1, c2, c3 = (int(v) for v in line.split())
    out = torch.zeros(4, dtype=torch.int32)
    k[(1,)](out, seed, c0, c1, c2, c3)
    print(*[int(v) & 0xFFFFFFFF for v in out])
"""


def test_philox4x32_matches_triton_library_generator():
    """Triton's `tl.philox` is an independent Philox4x32-10 (64-bit seed = key, four
    32-bit counter words); its CPU interpreter runs without a GPU."""
    rng = np.random.default_rng(3)
    cases = [(int(rng.integers(0, 2**62)), *[int(v) for v in rng.integers(0, 2**31, 4)]) for _ in range(6)]
    cases.append((0, 0, 0, 0, 0))
    try:
        res = subprocess.run([sys.executable, "-c", _TRITON_SNIPPET],
                             input="\n".join(" ".join(map(str, c)) for c in cases),
                             capture_output=True, text=True, timeout=600)
    except subprocess.TimeoutExpired:
        pytest.skip("triton interpreter timed out")
    if res.returncode != 0:
        pytest.skip("triton interpreter unavailable: " + res.stderr[-300:])
    lines = [ln for ln in res.stdout.strip().splitlines() if ln.strip()]
    assert len(lines) == len(cases)
    for (seed, c0, c1, c2, c3), ln in zip(cases, lines):
        want = [int(v) for v in ln.split()]
        got = [int(w) for w in philox4x32_10(seed & 0xFFFFFFFF, seed >> 32, c0, c1, c2, c3)]
        assert got == want


# --------------------------------------------------------------------------- GRBS (Definition 2)
@pytest.mark.parametrize("R", [1, 4, 32, 256, 1024])
def test_grbs_fraction_is_about_one_over_R(R):
    B = 99_833
    for t in (1, 2, 77):
        for stream in (STREAM_GRAD, STREAM_RESET):
            cnt = int(grbs_mask(0, t, stream, B, R).sum())
            sd = np.sqrt(B * (1 / R) * (1 - 1 / R))
            assert abs(cnt - B / R) <= 5 * sd + 1e-9
    if R == 1:
        assert grbs_mask(5, 9, 0, 1000, 1).all()


def test_grbs_is_a_pure_function_and_streams_steps_are_independent():
    B, R = 65_536, 4
    a = grbs_mask(7, 3, STREAM_GRAD, B, R)
    assert np.array_equal(a, grbs_mask(7, 3, STREAM_GRAD, B, R))
    for other in (grbs_mask(7, 3, STREAM_RESET, B, R), grbs_mask(7, 4, STREAM_GRAD, B, R),
                  grbs_mask(8, 3, STREAM_GRAD, B, R), grbs_mask(7 + 2**32, 3, STREAM_GRAD, B, R),
                  grbs_mask(7, 3 + 2**32, STREAM_GRAD, B, R)):
        both = int((a & other).sum())          # independent => about B/R^2
        assert abs(both - B / R**2) <= 5 * np.sqrt(B / R**2)
    # a slab of blocks with global ids is the slab of the global mask
    assert np.array_equal(grbs_mask(7, 3, 0, 100, R, block_begin=500), a[500:600])


def test_grbs_per_block_frequency_over_steps():
    B, R, T = 512, 8, 4000
    freq = np.zeros(B)
    for t in range(1, T + 1):
        freq += grbs_mask(11, t, STREAM_GRAD, B, R)
    z = (freq - T / R) / np.sqrt(T * (1 / R) * (1 - 1 / R))
    assert np.abs(z).max() < 5.0
    chi2 = float((z**2).sum())                  # ~ chi-square with B dof
    assert abs(chi2 - B) < 6 * np.sqrt(2 * B)


def test_grbs_is_a_one_over_R_approximate_compressor_in_expectation():
    """Definition 1 with delta = 1/R: E||C(v) - v||^2 = (1 - 1/R) ||v||^2."""
    d, bs, R = 10_000, 16, 4
    B = n_blocks(d, bs)
    v = np.random.default_rng(5).standard_normal(d)
    blk = np.arange(d) // bs
    ratios = []
    for t in range(1, 801):
        sel = grbs_mask(3, t, STREAM_GRAD, B, R)[blk] != 0
        ratios.append(((np.where(sel, v, 0) - v) ** 2).sum() / (v**2).sum())
    assert abs(np.mean(ratios) - (1 - 1 / R)) < 0.01


# --------------------------------------------------------------------------- helpers
def _run(cls, g_seq, x0, dtype=np.float64, masks=None, **kw):
    n, d = g_seq[0].shape
    o = cls(d, n, kw.pop("bs"), kw.pop("R1"), kw.pop("R2"), kw.pop("H"), kw.pop("eta"), kw.pop("beta"),
            kw.pop("seed", 0), dtype=dtype)
    o.set_x0(x0)
    for t, g in enumerate(g_seq, start=1):
        if masks is not None:
            o.inject_masks(*masks[t - 1])
        o.step(g)
    return o


def _rand_problem(seed, n, d, T):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d).astype(np.float32)
    g = [(rng.standard_normal(d)[None, :] + 0.5 * rng.standard_normal((n, d))).astype(np.float32)
         for _ in range(T)]
    return x0, g


# --------------------------------------------------------------------------- PSync (Algorithm 3)
def test_psync_identity_and_zero_compressors():
    rng = np.random.default_rng(0)
    v = rng.standard_normal((5, 12))
    vp, r = psync(v, np.ones(12, bool))                   # C = identity: plain average, no residual
    assert np.allclose(vp, v.mean(0)[None, :].repeat(5, 0), rtol=0, atol=1e-15) and not r.any()
    vp, r = psync(v, np.zeros(12, bool))                  # C = 0: nothing is exchanged
    assert np.array_equal(vp, v) and np.array_equal(r, v)
    sel = np.arange(12) % 3 == 0                          # mixed: mean of v' over workers == mean of v
    vp, r = psync(v, sel)
    assert np.allclose(vp.mean(0), v.mean(0), atol=1e-15)
    assert np.array_equal(r[:, sel], np.zeros((5, int(sel.sum())))) and np.array_equal(r[:, ~sel], v[:, ~sel])


# --------------------------------------------------------------------------- R = 1: synchronous SGD
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_R1_reduces_to_synchronous_sgd_bit_exact(dtype):
    """Identity compressors: every worker applies eta * mean(g) (Table 2's R_C = 1 column is SGD)."""
    n, d, T, eta = 8, 300, 12, 0.1
    x0, g = _rand_problem(10, n, d, T)
    o = _run(CSEROracle, g, x0, dtype, bs=16, R1=1, R2=1, H=3, eta=eta, beta=0.0)
    x = x0.astype(dtype)
    eta_t = dtype(np.float32(eta))
    for gt in g:                                          # textbook loop
        s = (eta_t * gt[0].astype(dtype))
        for i in range(1, n):
            s = s + eta_t * gt[i].astype(dtype)
        x = x - s / dtype(n)
    for i in range(n):
        assert np.array_equal(o.x[i], x)
    assert not o.e.any()


def test_R1_with_momentum_is_nesterov_momentum_sgd_on_the_mean_gradient():
    """Section 3.2: m_t = beta m_{t-1} + g_t, x_t = x_{t-1} - eta (beta m_t + g_t)."""
    n, d, T, eta, beta = 4, 200, 25, 0.1, 0.9
    x0, g = _rand_problem(11, n, d, T)
    o = _run(CSEROracle, g, x0, np.float64, bs=8, R1=1, R2=1, H=4, eta=eta, beta=beta)
    eta_t, beta_t = float(np.float32(eta)), float(np.float32(beta))
    x, M = x0.astype(np.float64), np.zeros(d)
    for gt in g:
        gbar = gt.astype(np.float64).mean(0)
        M = beta_t * M + gbar
        x = x - eta_t * (beta_t * M + gbar)
    assert np.allclose(o.x, x[None, :], rtol=1e-12, atol=1e-12)
    assert np.abs(o.x - o.x[0]).max() == 0 and not o.e.any()


# --------------------------------------------------------------------------- hand example
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("beta", [0.0, 0.5])
def test_hand_worked_example(beta, dtype):
    gold = read_hand_example()
    g = [np.array([[1, 2, -1, 0], [3, -2, 1, 4]], np.float32), np.array([[2, 2, 2, 2], [0, 4, -2, 6]], np.float32)]
    masks = [([1, 0], None), ([0, 1], [0, 1])]
    o = CSEROracle(4, 2, 2, 7, 7, 2, 0.5, beta, 0, dtype=dtype)
    o.set_x0([1, 2, 3, 4])
    for t in (1, 2):
        o.inject_masks(*masks[t - 1])
        o.step(g[t - 1])
        for name in ("x", "e") + (("m",) if beta else ()):
            for i in range(2):
                assert np.array_equal(getattr(o, name)[i], np.array(gold[(beta, t, name, i)], dtype)), (t, name, i)


# --------------------------------------------------------------------------- closed form, exact rationals
def _closed_form(x0, g_seq, masks, H, eta, beta, bs):
    """Non-iterative expansion: m from Lemma 4's sum, e as minus the sum of the residual updates
    since the block's last reset, mean model from x-bar_t - x-bar_{t-1} = -mean_i p_{i,t}, and
    x_i = x-bar + e_i - mean_k e_k (Lemma 1)."""
    T = len(g_seq)
    n, d = len(g_seq[0]), len(g_seq[0][0])
    F = Fraction
    p = [[[None] * d for _ in range(n)] for _ in range(T)]
    m_T = [[None] * d for _ in range(n)]
    for i in range(n):
        for j in range(d):
            for tau in range(1, T + 1):
                m = sum(F(beta) ** (tau - s) * F(g_seq[s - 1][i][j]) for s in range(1, tau + 1)) if beta else F(0)
                p[tau - 1][i][j] = F(eta) * (F(beta) * m + F(g_seq[tau - 1][i][j]))
                if tau == T:
                    m_T[i][j] = m
    x = [[None] * d for _ in range(n)]
    e = [[None] * d for _ in range(n)]
    for j in range(d):
        b = j // bs
        tau0 = 0
        for tau in range(1, T + 1):
            if tau % H == 0 and masks[tau - 1][1][b]:
                tau0 = tau
        for i in range(n):
            e[i][j] = -sum((1 - masks[tau - 1][0][b]) * p[tau - 1][i][j] for tau in range(tau0 + 1, T + 1))
        xbar = F(x0[j]) - sum(sum(p[tau][i][j] for i in range(n)) / n for tau in range(T))
        ebar = sum(e[i][j] for i in range(n)) / n
        for i in range(n):
            x[i][j] = xbar + e[i][j] - ebar
    return x, e, m_T


@pytest.mark.parametrize("beta", [0.0, 0.5])
@pytest.mark.parametrize("n,H", [(2, 2), (4, 3), (8, 1)])
def test_closed_form_in_exact_rational_arithmetic(beta, n, H):
    rng = np.random.default_rng(100 + n + H)
    d, bs, T, eta = 11, 3, 7, 0.25                       # ragged last block (2 of 3)
    B = n_blocks(d, bs)
    x0 = rng.integers(-8, 9, d) / 4.0
    g = [rng.integers(-8, 9, (n, d)) / 8.0 for _ in range(T)]
    masks = [(rng.integers(0, 2, B).tolist(), rng.integers(0, 2, B).tolist()) for _ in range(T)]
    o = _run(CSEROracle, [gt.astype(np.float32) for gt in g], x0, np.float64, masks=masks,
             bs=bs, R1=2, R2=2, H=H, eta=eta, beta=beta)
    x, e, m = _closed_form(x0.tolist(), [gt.tolist() for gt in g], masks, H, eta, beta, bs)
    for i in range(n):
        for j in range(d):
            assert Fraction(float(o.x[i, j])) == x[i][j], ("x", i, j)
            assert Fraction(float(o.e[i, j])) == e[i][j], ("e", i, j)
            if beta:
                assert Fraction(float(o.m[i, j])) == m[i][j], ("m", i, j)
    # dyadic inputs: Lemma 1 holds with no rounding at all
    assert np.abs((o.x - o.e) - (o.x - o.e)[0]).max() == 0


# --------------------------------------------------------------------------- invariants with real GRBS draws
@pytest.mark.parametrize("beta", [0.0, 0.9])
def test_lemma1_mean_model_identity_and_reset_zeroes(beta):
    n, d, T, bs, R1, R2, H, eta = 8, 2000, 40, 16, 4, 2, 4, 0.1
    x0, g = _rand_problem(20, n, d, T)
    o = CSEROracle(d, n, bs, R1, R2, H, eta, beta, 42)
    o.set_x0(x0)
    eta_t, beta_t = float(np.float32(eta)), float(np.float32(beta))
    m = np.zeros((n, d))
    xbar = x0.astype(np.float64)
    blk = np.arange(d) // bs
    saw_reset_sel = False
    for gt in g:
        o.step(gt)
        if beta:
            m = beta_t * m + gt
            p = eta_t * (beta_t * m + gt)
        else:
            p = eta_t * gt.astype(np.float64)
        xbar = xbar - p.mean(0)                               # uncompressed (momentum) SGD on the mean
        assert np.allclose(o.x.mean(0), xbar, rtol=0, atol=1e-12)
        diff = (o.x - o.e) - (o.x - o.e)[0]                   # Lemma 1
        assert np.abs(diff).max() < 1e-12
        if o.t % H == 0:
            sel = o.mask_r[blk] != 0
            saw_reset_sel |= bool(sel.any())
            assert not o.e[:, sel].any()                      # error is reset to exactly zero
            assert np.abs(o.x[:, sel] - o.x[0, sel]).max() < 1e-12   # so local models agree there
            assert o.e[:, ~sel].any()
    assert saw_reset_sel
    if beta:
        assert np.allclose(o.m, m, rtol=1e-13, atol=1e-13)    # m_t = sum beta^(t-tau) g_tau


def test_momentum_closed_form_sum():
    n, d, T, beta = 3, 50, 15, 0.9
    x0, g = _rand_problem(21, n, d, T)
    o = _run(CSEROracle, g, x0, bs=8, R1=4, R2=4, H=5, eta=0.1, beta=beta)
    b = float(np.float32(beta))
    want = sum(b ** (T - tau) * g[tau - 1].astype(np.float64) for tau in range(1, T + 1))
    assert np.allclose(o.m, want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("beta", [0.0, 0.9])
def test_single_worker_is_plain_sgd_whatever_the_compressors(beta):
    d, T, eta = 500, 30, 0.05
    x0, g = _rand_problem(22, 1, d, T)
    o = _run(CSEROracle, g, x0, bs=8, R1=16, R2=4, H=3, eta=eta, beta=beta)
    eta_t, beta_t = float(np.float32(eta)), float(np.float32(beta))
    x, m = x0.astype(np.float64), np.zeros(d)
    for gt in g:
        m = beta_t * m + gt[0]
        x = x - eta_t * ((beta_t * m + gt[0]) if beta else gt[0].astype(np.float64))
    assert np.allclose(o.x[0], x, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("beta", [0.0, 0.9])
def test_implementation_II_gives_the_same_models(beta):
    n, d, T = 8, 1500, 48
    x0, g = _rand_problem(23, n, d, T)
    kw = dict(bs=32, R1=4, R2=2, H=4, eta=0.1, beta=beta, seed=9)
    a = _run(CSEROracle, g, x0, **kw)
    b = _run(CSERImpl2Oracle, g, x0, **kw)
    assert np.allclose(a.x, b.x, rtol=1e-12, atol=1e-12)
    if beta:
        assert np.array_equal(a.m, b.m)


def test_partial_local_sgd_with_full_reset_is_local_sgd():
    """C2 = 0 (nothing exchanged per step) and delta_1 = 1: H local steps, then plain averaging."""
    n, d, T, H, eta = 4, 64, 12, 4, 0.1
    x0, g = _rand_problem(24, n, d, T)
    B = n_blocks(d, 8)
    masks = [([0] * B, [1] * B) for _ in range(T)]
    o = _run(CSEROracle, g, x0, masks=masks, bs=8, R1=1, R2=1, H=H, eta=eta, beta=0.0)
    x = np.repeat(x0.astype(np.float64)[None, :], n, 0)
    for t, gt in enumerate(g, 1):
        x = x - float(np.float32(eta)) * gt.astype(np.float64)
        if t % H == 0:
            x[:] = x.mean(0)
    assert np.allclose(o.x, x, rtol=1e-12, atol=1e-12)


def test_column_subset_evaluation_equals_full_evaluation():
    n, d, T, bs = 4, 700, 9, 32
    x0, g = _rand_problem(25, n, d, T)
    full = _run(CSEROracle, g, x0, np.float32, bs=bs, R1=4, R2=2, H=3, eta=0.1, beta=0.9, seed=5)
    cols = np.r_[0:32, 96:160, 672:700]
    sub = CSEROracle(d, n, bs, 4, 2, 3, 0.1, 0.9, 5, dtype=np.float32, cols=cols)
    sub.set_x0(x0[cols])
    for gt in g:
        sub.step(gt[:, cols])
    for name in "xem":
        assert np.array_equal(getattr(sub, name), getattr(full, name)[:, cols])


def test_float32_evaluation_stays_within_the_stated_tolerances_of_float64():
    """1e-6 relative + 1e-7 absolute after one step; 1e-4 relative after 100 steps."""
    n, d, T = 8, 4096, 100
    x0, g = _rand_problem(26, n, d, T)
    kw = dict(d=d, n_workers=n, block_size=64, R1=4, R2=4, H=4, eta=0.1, beta=0.9, seed=1)
    a, b = CSEROracle(dtype=np.float32, **kw), CSEROracle(dtype=np.float64, **kw)
    a.set_x0(x0), b.set_x0(x0)
    for t, gt in enumerate(g, 1):
        a.step(gt), b.step(gt)
        if t == 1:
            for name in "xem":
                u, v = getattr(a, name).astype(np.float64), getattr(b, name)
                assert (np.abs(u - v) <= 1e-6 * np.abs(v) + 1e-7).all()
    for name in "xem":
        u, v = getattr(a, name).astype(np.float64), getattr(b, name)
        rms = np.sqrt((v**2).mean())
        assert (np.abs(u - v) <= 1e-4 * np.abs(v) + 1e-4 * rms).all()
        assert np.abs(u - v).max() <= 1e-5 * np.abs(v).max()


# --------------------------------------------------------------------------- C2 = 0 special cases (Appendix A.1)
def test_ratio_zero_means_the_compressor_keeps_nothing():
    assert not grbs_mask(3, 5, STREAM_GRAD, 1000, 0).any()


def test_csea_is_cser_with_no_update_sync_and_reset_every_step():
    n, d, T = 4, 600, 20
    x0, g = _rand_problem(30, n, d, T)
    a = _run(CSEROracle, g, x0, bs=8, R1=0, R2=4, H=1, eta=0.1, beta=0.0, seed=13)
    c = CSEAOracle(d, n, 8, 4, 0.1, 13)
    c.set_x0(x0)
    for gt in g:
        c.step(gt)
        assert not c.e[:, c.mask_r[c.block_of_col] != 0].any()
    assert np.allclose(a.x, c.x, rtol=1e-12, atol=1e-12) and np.allclose(a.e, c.e, rtol=1e-12, atol=1e-12)
    assert np.abs(a.x - a.x[0]).max() > 1e-3            # local models do bifurcate


def test_cser_pl_with_identity_reset_compressor_is_local_sgd():
    """C2 = 0 drawn natively (R1 = 0) and delta_1 = 1 (R2 = 1): local SGD with period H."""
    n, d, T, H, eta = 4, 64, 12, 4, 0.1
    x0, g = _rand_problem(31, n, d, T)
    o = _run(CSEROracle, g, x0, bs=8, R1=0, R2=1, H=H, eta=eta, beta=0.0)
    x = np.repeat(x0.astype(np.float64)[None, :], n, 0)
    for t, gt in enumerate(g, 1):
        x = x - float(np.float32(eta)) * gt.astype(np.float64)
        if t % H == 0:
            x[:] = x.mean(0)
    assert np.allclose(o.x, x, rtol=1e-12, atol=1e-12)
    assert not o.mask_g.any()


# --------------------------------------------------------------------------- exact-count GRBS (Definition 2, literal)
def test_exact_count_selects_exactly_round_B_over_R_blocks():
    for B, R in ((4096, 4), (69_822, 32), (24_959, 256), (99_833, 1024), (163_644, 64), (10, 3), (3, 16), (7, 1), (5, 0)):
        k = exact_count(B, R)
        assert k == (0 if R == 0 else min(B, int(np.floor(B / R + 0.5))))
        for t in (1, 2, 9):
            for stream in (STREAM_GRAD, STREAM_RESET):
                assert int(grbs_mask_exact(1, t, stream, B, R).sum()) == k


def test_exact_count_is_the_k_smallest_draws_by_brute_force():
    from oracle import philox4x32_10
    B, R, seed, t = 37, 5, 99, 3
    words = [int(philox4x32_10(seed, 0, b, t, 0, STREAM_RESET)[0]) for b in range(B)]
    chosen = sorted(range(B), key=lambda b: (words[b], b))[: exact_count(B, R)]
    want = np.zeros(B, np.uint8)
    want[chosen] = 1
    assert np.array_equal(grbs_mask_exact(seed, t, STREAM_RESET, B, R), want)
    # whatever is selected has a draw no larger than whatever is not
    m = grbs_mask_exact(seed, t, STREAM_RESET, B, R).astype(bool)
    assert max(w for w, s in zip(words, m) if s) <= min(w for w, s in zip(words, m) if not s)


def test_exact_count_marginals_are_uniform_and_delta_is_k_over_B():
    B, R, T = 256, 8, 3000
    k = exact_count(B, R)
    freq = np.zeros(B)
    v = np.random.default_rng(6).standard_normal(B * 4)
    blk = np.arange(B * 4) // 4
    ratios = []
    for t in range(1, T + 1):
        m = grbs_mask_exact(21, t, STREAM_GRAD, B, R)
        freq += m
        if t <= 600:
            sel = m[blk] != 0
            ratios.append(((np.where(sel, v, 0) - v) ** 2).sum() / (v**2).sum())
    z = (freq - T * k / B) / np.sqrt(T * (k / B) * (1 - k / B))
    assert np.abs(z).max() < 5.0
    assert abs(np.mean(ratios) - (1 - k / B)) < 0.01


def test_exact_count_mode_keeps_the_invariants():
    n, d, T = 4, 640, 24
    x0, g = _rand_problem(40, n, d, T)
    o = CSEROracle(d, n, 8, 4, 2, 3, 0.1, 0.9, 5, exact_count=True)
    o.set_x0(x0)
    xbar = x0.astype(np.float64)
    m = np.zeros((n, d))
    for gt in g:
        o.step(gt)
        m = float(np.float32(0.9)) * m + gt
        xbar = xbar - (float(np.float32(0.1)) * (float(np.float32(0.9)) * m + gt)).mean(0)
        assert int(o.mask_g.sum()) == exact_count(o.B, 4)
        assert np.allclose(o.x.mean(0), xbar, atol=1e-12)
        assert np.abs((o.x - o.e) - (o.x - o.e)[0]).max() < 1e-12


# --------------------------------------------------------------------------- Lemma 3 (error after a reset is bounded)
def test_error_after_reset_stays_below_the_bound_of_lemma_3():
    """E||e_{i,t}||^2 <= (1 - d2)(1 - d1) eta^2 H^2 V2 / (1 - sqrt(1 - d1))^2 at every t with t mod H = 0,
    with d2 = 1/R1 (update compressor), d1 = 1/R2 (reset compressor) and V2 >= E||g||^2."""
    n, d, bs, R1, R2, H, eta, T = 4, 512, 8, 4, 2, 4, 0.1, 40
    d1, d2 = 1.0 / R2, 1.0 / R1
    sq = {t: [] for t in range(H, T + 1, H)}
    g_sq = []
    for seed in range(30):
        rng = np.random.default_rng(1000 + seed)
        o = CSEROracle(d, n, bs, R1, R2, H, eta, 0.0, seed)
        o.set_x0(rng.standard_normal(d))
        for t in range(1, T + 1):
            g = rng.standard_normal((n, d))
            g_sq.append((g**2).sum(1).mean())
            o.step(g)
            if t % H == 0:
                sq[t].append((o.e**2).sum(1).mean())
    V2 = float(np.mean(g_sq))
    bound = (1 - d2) * (1 - d1) * float(np.float32(eta)) ** 2 * H**2 * V2 / (1 - np.sqrt(1 - d1)) ** 2
    worst = max(float(np.mean(v)) for v in sq.values())
    assert 0 < worst <= bound
    assert worst > 1e-3 * bound            # the bound is loose but not vacuous for this setting
