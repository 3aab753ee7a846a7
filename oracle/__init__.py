"""CPU oracle for the OrbitQuant quantized-linear hot path.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the hot path computes, written from the paper's equations.  It shares no
code, tables or constants with the CUDA library and must never be imported by
the product path: only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it.

Modules
-------
bf16      bit-level bfloat16 <-> float conversions (round-to-nearest-even)
rpbh      randomized permuted block-Hadamard rotation (Eq. 9), dense definition
codebook  Lloyd-Max scalar codebook for the sphere-coordinate marginal (Eq. 2-3)
quantize  per-row rotate -> norm -> nearest centroid (Eq. 4-8, Algorithm 1)
qlinear   product of the decoded operands with both norms re-attached
adaln     AdaLN modulation projection: weight-only INT4 round-to-nearest in groups of 64, bf16 activations

Parity pins: every function here is pinned by tests/test_oracle_*.py against
closed forms, exact invariants, brute force and classical published tables.
"""
