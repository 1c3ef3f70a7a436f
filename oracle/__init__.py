"""ORACLE — TEST INFRASTRUCTURE ONLY.

Plain, slow, fp64 CPU statement of what the PuzzleKV hot path computes, written
from the paper.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may import this package; the product (the CUDA library and its binding)
never does, and this package never imports the product.

Modules
-------
svd         per-page truncated SVD (Eq. 2) by one-sided Jacobi (C, fp64)
attention   softmax attention: the plain definition (Eq. 1) and the page-wise
            factor form with online-softmax merge (Eq. 4, Eq. 5)
cache       the hybrid paged cache state machine (Section 3.3: construction,
            mixed attention, incremental update)
quant       INT4 quantization of the factors (Section 4.3)
bf16        bf16 storage rounding of factors (integer arithmetic on bit patterns)
accounting  storage-ratio and size formulas (Eq. 3, Section 1)

Parity status: every function here is pinned by tests/test_oracle_*.py against
values printed in the paper, closed forms, library routines or brute force.
"""
