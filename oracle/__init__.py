"""CPU oracle -- TEST INFRASTRUCTURE ONLY.

Slow, plain restatements of what the 2M / Ozaki-II complex-GEMM path computes, written from
the paper and independent of the CUDA library (no shared code, tables or constants).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product path never does.

  oracle.direct : the 4M definitions (exact integer product; double-double complex product)
  oracle.staged : Algorithm 1 ("2M Ozaki-II") step by step in arbitrary-precision integers
"""
