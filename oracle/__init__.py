"""CPU oracle for the reversible residual network hot path (float64).

TEST INFRASTRUCTURE ONLY.  The oracle is a plain, slow, obviously-correct
restatement of what the paper defines: BN->ReLU->conv residual functions
(Section 2.2, Eq. 2), the reversible block and its inverse (Section 3.1),
ordinary stored-activation backprop (Section 2.1, Eq. 1) and the
activation-reconstructing backprop (Algorithm 1), plus the stored
non-reversible layers of a classification stack (Section 3.1-3.2).

Only tests, the smoke check and the timed CPU-baseline leg of the benchmark
may import it.  It shares no code with the CUDA path and imports nothing from
the product package.

Parity status: every function is pinned by invariants the paper states
(exact invertibility, Algorithm 1 == ordinary backprop), by central finite
differences, by closed forms, and by an independent float64 autograd
cross-check.  The paper prints no worked numeric example, so no activation or
gradient VALUE is pinned to a printed number.
"""
