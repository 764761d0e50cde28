"""CPU oracle for the CSER / M-CSER optimizer step (test infrastructure, not product).

This package is a plain, slow restatement of the paper's algorithms in NumPy:

* ``philox``  - the Philox4x32-10 counter-based generator (Salmon et al., SC'11)
* ``grbs``    - the globally-randomized blockwise sparsifier mask (Definition 2)
* ``cser``    - PSync (Algorithm 3), Get_p (Appendix A.4), CSER (Algorithm 2),
                M-CSER implementation I (Algorithm 4) and the memory-saving
                implementation II (Appendix A.4) and the special case CSEA (Appendix A.1)

It exists only so that tests, the smoke check and the benchmark's CPU-baseline
leg can compare the CUDA library against something that can be checked against
the paper by eye.  It shares no code with the CUDA path, never imports the
product package, and the product never imports it.  Every function is pinned
by the CPU test-suite to facts the paper or the mathematics fix (special cases
that reduce to textbook SGD, Lemma 1, the mean-model identity, closed forms,
exact rational brute force, library generators); none is "parity unpinned".
"""
from .philox import philox4x32_10, philox4_generic          # noqa: F401
from .grbs import grbs_mask, grbs_mask_exact, exact_count, n_blocks, STREAM_GRAD, STREAM_RESET   # noqa: F401
from .cser import psync, get_p, CSEROracle, CSERImpl2Oracle, CSEAOracle  # noqa: F401
