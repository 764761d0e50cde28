"""CSER / M-CSER optimizer step, written out literally (oracle side).

Test infrastructure only.  n simulated workers hold rows of [n, k] arrays; the
mean over the worker axis stands in for the allreduce.  The code follows the
paper's algorithms in their own order and notation, materialising PSync's
intermediate vectors v', r and v-bar':

* ``psync``            - Algorithm 3 (partial synchronization)
* ``get_p``            - Appendix A.4, "Calculate update on worker i"
* ``CSEROracle``       - Algorithm 2 (beta = 0) and Algorithm 4 (beta != 0)
* ``CSERImpl2Oracle``  - Appendix A.4, implementation II (no error array)
* ``CSEAOracle``       - Appendix A.1, CSEA (implementation I), the special case C2 = 0, H = 1

Arithmetic runs in ``dtype``: float64 (default) is the reference trajectory;
float32 evaluates the same expressions in the storage precision, one IEEE
operation per NumPy call (no fused multiply-add), sums over workers in
ascending worker order starting from worker 0's value, mean = sum / n.

Readings taken where the paper is silent or inconsistent:

* R1 is the ratio of the compressor applied to the update every step
  (Algorithm 2 line 6), R2 the ratio of the compressor applied to the error
  every H steps (line 11).
* With no momentum the update is p = eta * g formed before PSync (Get_p), not
  eta * mean(g).
* On a reset step, line 12 (x <- x - e + e') changes only the reset-selected
  blocks; elsewhere e' = e and the line is the identity, so x is left as is.
* The two masks of a reset step are drawn independently.
* ``exact_count=True`` switches the masks to the literal reading of Definition 2
  (exactly round(B/R) blocks, see ``grbs.grbs_mask_exact``).
* eta and beta are the float32 values an `float` ABI argument would carry.

The oracle may be evaluated on any subset of columns (``cols``): columns are
independent given the masks, which always use global block ids.
"""
import numpy as np
from .grbs import grbs_mask, grbs_mask_exact, n_blocks, STREAM_GRAD, STREAM_RESET


def _mean_over_workers(vc):
    """(vc[0] + vc[1] + ... + vc[n-1]) / n, ascending, in vc's dtype."""
    acc = vc[0].copy()
    for i in range(1, vc.shape[0]):
        acc = acc + vc[i]
    return acc / vc.dtype.type(vc.shape[0])


def psync(v, sel):
    """Algorithm 3.  v: [n, k]; sel: bool[k], the columns the compressor keeps.

    Returns (v'_i, r_i) with v'_i = mean_k C(v_k) + r_i and r_i = v_i - C(v_i).
    """
    v_c = np.where(sel[None, :], v, v.dtype.type(0))      # line 4: v' = C(v)
    r = v - v_c                                           # line 5
    v_bar = _mean_over_workers(v_c)                       # line 7
    return v_bar[None, :] + r, r                          # line 8


def get_p(m, g, eta, beta):
    """Appendix A.4 Get_p.  Returns (p, m_new); m is None when beta == 0."""
    if beta != 0:
        m = beta * m + g
        p = eta * (beta * m + g)
    else:
        p = eta * g
    return p, m


class _Base:
    def __init__(self, d, n_workers, block_size, R1, R2, H, eta, beta, seed,
                 dtype=np.float64, cols=None, exact_count=False):
        self._draw = grbs_mask_exact if exact_count else grbs_mask
        self.d, self.n, self.bs = int(d), int(n_workers), int(block_size)
        self.R1, self.R2, self.H = int(R1), int(R2), int(H)
        self.seed = int(seed)
        self.dtype = np.dtype(dtype)
        T = self.dtype.type
        self.eta = T(np.float32(eta))
        self.beta = T(np.float32(beta))
        self.B = n_blocks(self.d, self.bs)
        self.cols = np.arange(self.d, dtype=np.int64) if cols is None else np.asarray(cols, dtype=np.int64)
        self.block_of_col = self.cols // self.bs
        k = self.cols.size
        self.t = 0
        self.x = np.zeros((self.n, k), self.dtype)
        self.m = np.zeros((self.n, k), self.dtype) if self.beta != 0 else None
        self.mask_g = np.zeros(self.B, np.uint8)
        self.mask_r = np.zeros(self.B, np.uint8)
        self._injected = None

    def set_x0(self, x0):
        """x_{i,0} = x0 for every worker (x0 holds the entries at ``cols``); t = 0."""
        self.x[:] = np.asarray(x0, self.dtype)[None, :]
        if self.m is not None:
            self.m[:] = 0
        self.t = 0

    def inject_masks(self, mask_g, mask_r=None):
        """Use these block masks instead of GRBS draws for the next step only."""
        self._injected = (np.asarray(mask_g, np.uint8),
                          None if mask_r is None else np.asarray(mask_r, np.uint8))

    def _masks(self, t, is_reset):
        if self._injected is not None:
            mg, mr = self._injected
            self._injected = None
            self.mask_g = mg
            if is_reset:
                self.mask_r = mr
        else:
            self.mask_g = self._draw(self.seed, t, STREAM_GRAD, self.B, self.R1)
            if is_reset:
                self.mask_r = self._draw(self.seed, t, STREAM_RESET, self.B, self.R2)
        sel_g = self.mask_g[self.block_of_col] != 0
        sel_r = (self.mask_r[self.block_of_col] != 0) if is_reset else None
        return sel_g, sel_r


class CSEROracle(_Base):
    """Algorithm 2 (beta == 0) / Algorithm 4 (beta != 0), implementation I."""

    def __init__(self, *a, **kw):
        super().__init__(*a, **kw)
        self.e = np.zeros_like(self.x)

    def set_x0(self, x0):
        super().set_x0(x0)
        self.e[:] = 0

    def step(self, g):
        """One iteration t <- t + 1 on gradients g [n, k] (columns ``cols``)."""
        g = np.asarray(g, self.dtype)
        self.t += 1
        is_reset = self.t % self.H == 0
        sel_g, sel_r = self._masks(self.t, is_reset)
        p, self.m = get_p(self.m, g, self.eta, self.beta)          # Alg. 4 lines 6-7
        p_prime, r = psync(p, sel_g)                               # line 8
        self.x = self.x - p_prime                                  # line 9
        self.e = self.e - r
        if is_reset:
            e_prime, e_new = psync(self.e, sel_r)                  # line 13
            self.x = np.where(sel_r[None, :], (self.x - self.e) + e_prime, self.x)   # line 14
            self.e = e_new


class CSERImpl2Oracle(_Base):
    """Appendix A.4, CSER implementation II: no error array; on a reset step the
    partial synchronization is applied to the local models themselves."""

    def step(self, g):
        g = np.asarray(g, self.dtype)
        self.t += 1
        is_reset = self.t % self.H == 0
        sel_g, sel_r = self._masks(self.t, is_reset)
        p, self.m = get_p(self.m, g, self.eta, self.beta)
        p_prime, _ = psync(p, sel_g)
        self.x = self.x - p_prime
        if is_reset:
            self.x, _ = psync(self.x, sel_r)


class CSEAOracle(_Base):
    """Appendix A.1, "CSEA (Implementation I)": SGD with error assimilation, the special case
    of CSER with C2 = 0 and H = 1, in the paper's own three-line form (no momentum):
        p_i  <- e_i - eta * g_i
        e'_i, e_i <- PSync(p_i, C1)
        x_i  <- x_i + e'_i - e_{i,t-1}
    The last line is applied to the whole vector, as printed."""

    def __init__(self, d, n_workers, block_size, R2, eta, seed, dtype=np.float64, cols=None):
        super().__init__(d, n_workers, block_size, 0, R2, 1, eta, 0.0, seed, dtype=dtype, cols=cols)
        self.e = np.zeros_like(self.x)

    def step(self, g):
        g = np.asarray(g, self.dtype)
        self.t += 1
        self.mask_r = grbs_mask(self.seed, self.t, STREAM_RESET, self.B, self.R2)
        sel = self.mask_r[self.block_of_col] != 0
        e_old = self.e
        p = e_old - self.eta * g
        e_prime, self.e = psync(p, sel)
        self.x = self.x + e_prime - e_old
