"""CPU FP64 oracle for Generalized PolyDot coded matrix multiplication.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, written-for-reading
restatement of what the paper's method computes (arXiv 1811.10751).  It exists so
that tests can check the CUDA library element by element, and so that the
benchmark can time a CPU baseline.  It shares no code with the CUDA library and
must never be imported by it; the library has no CPU fallback.

Modules
    code    : block partition, encoding polynomials, thresholds, parity-check matrix
    product : encode / worker products / interpolation decode / coded update
    locate  : Algorithm 1 at node level (exhaustive form and subspace form)
    inject  : seeded soft-error injection (counter-based SplitMix64)
    dnn     : uncoded FP64 SGD steps and the coded layer step built from the above

Parity pins (tests/test_oracle_*.py): thresholds against the numbers printed in the
paper's worked examples and theorems and against brute-force exponent counting;
decoded product against the uncoded product and against exact rational Lagrange
interpolation; every threshold-sized subset decoding to the same result; the
parity-check matrix against the closed divided-difference form; the locator
against exhaustive search and the three claims of Theorem 3; the coded update
against Eq. (10); DNN gradients against finite differences.

Parity unpinned: the numeric zero-tolerances of the locator (tau_col, tau_in) and
the injector's magnitude ranges are engineering constants with no value in the
paper.
"""
