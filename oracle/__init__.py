"""CPU oracle for SpecHub / RRS / RRSw sampling-verification (arXiv 2411.05289).

TEST INFRASTRUCTURE ONLY.  A thin ctypes wrapper around ``spechub_oracle.c``
(plain C, fp64, single-threaded).  It shares nothing with the CUDA library:
only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  Every function cites the passage of the paper it follows in the
C source.

Parity pins (see ``tests/test_oracle_pins.py``): the worked example of the
captions of Figures 4 and 5, exactness of the emitted token's law (Theorem 2)
by enumeration for V <= 8, the closed form against a brute-force LP on
SpecHub's support (Section 3.2), hub mass = p(a) (Corollary 1), Theorem 3's
ordering against RRS, the T -> 0 top-2 limit (Section 5.2), and the
degenerate rows; ``cond`` (the conditioning figure the parity checker sizes its tolerance with)
against the derivatives of the oracle's own acceptance ratios (``tests/test_oracle_cond.py``).
``fanout`` runs the batch calls on several cores (same results, bit for bit).  Parity unpinned: the
printed digits of the paper's toy table only (``toy_table.py``).
"""
from .oracle import (  # noqa: F401
    NODE_DTYPE,
    STATUS_BITS,
    build,
    cdf_interval,
    draft_batch,
    hub,
    inv_cdf,
    rrs_draft,
    rrs_k_draft,
    rrs_k_draft_batch,
    rrs_k_residual,
    rrs_k_verify,
    rrs_k_verify_batch,
    rrs_residual,
    rrs_verify,
    softmax,
    spechub_draft,
    spechub_residual,
    spechub_verify,
    verify_batch,
    walk,
    walk_k,
)
